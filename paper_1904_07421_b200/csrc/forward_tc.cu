// Batched cell evaluation on the 5th-generation tensor cores (bf16 operands, fp32 accumulation in TMEM).
//
// Every dense contraction of the path is one instance of gemm_tc_kernel, a persistent, warp-specialised
// TMA -> shared memory -> tcgen05.mma -> TMEM -> epilogue pipeline, with the cell arithmetic fused into the
// epilogue so that no pre-activation of a leaf ever reaches memory:
//
//   EPI_XPROJ  Z = W x + b for all nodes at once (the leaf-independent input projection), rows in level order
//              (level_order_x_kernel lays x out that way in one pass).  Leaf tiles compute only the i, o, u blocks
//              and finish in the epilogue (c = sig(z_i) tanh(z_u), h = sig(z_o) tanh(c)); tiles of internal
//              nodes store their four pre-activations to P.
//   EPI_F      the per-child forget gates of one level.  The bf16 copy of h is kept in CHILD ORDER: the row of a
//              node sits at the slot of the edge that leads to it, edges numbered by (position of the parent in
//              level order, index in the parent's child list).  The children of a level's nodes are therefore one
//              contiguous range of rows, sorted by parent: the product U_f h_k over them is a plain GEMM with TMA
//              operands.  It is computed TRANSPOSED, hidden units along the accumulator rows and edges along its
//              columns, so that a thread owns one hidden unit and meets the edges of a parent one after the other:
//              the epilogue turns every value into f_jk c_k = sig(W_f x_j + b_f + U_f h_k) c_k and adds the values of
//              one parent up in a register, and only S_j = sum_k f_jk c_k, one row per PARENT, leaves the kernel.
//   EPI_LEVEL  one level: (i, o, u) pre-activations = P + U_iou h~ with h~ the child sums; the epilogue adds
//              S_j and finishes c_j = i u + S_j, h_j = o tanh(c_j), and files the bf16 copy of h_j at its slot.
//
// childsum_kernel produces the operand h~ of EPI_LEVEL: one warp per node adds the node's (contiguous) child rows.
// The level loop is host-driven here (three launches per level); forests whose levels are too small for that
// run the cooperative single-launch kernel of forward_small.cu instead.
#include <cuda.h>
#include <stdlib.h>

#include "common.cuh"
#include "ptx_sm100.cuh"

namespace jdb {

namespace {

using namespace ptx;

constexpr int BM = 128;
constexpr int BK = 64;
constexpr int STAGES = 4;
constexpr int MAX_BN = 256;
constexpr int A_BYTES = BM * BK * 2;
constexpr int B_BYTES_MAX = MAX_BN * BK * 2;
constexpr int STAGE_BYTES = A_BYTES + B_BYTES_MAX;
constexpr int GEMM1_THREADS = 224;  // warp 0: TMA producer, warps 1 and 6: MMA issuers, warps 2-5: epilogue
// The forget-gate GEMM's epilogue is instruction-bound (a segmented sum over the accumulator rows per 16-column
// step), and a scheduler with a single warp issues well below one instruction per cycle: it runs EIGHT epilogue
// warps, two per TMEM lane quarter and per scheduler, which take the steps of a tile alternately.
constexpr int GEMMF_THREADS = 320;  // warp 0: TMA producer, warp 1: MMA issuer, warps 2-9: epilogue
__host__ __device__ constexpr int gemm_threads(int epi) { return (epi == 2 || epi == 3) ? GEMMF_THREADS : GEMM1_THREADS; }
// the CTA-pair forget-gate GEMM runs sixteen epilogue warps (four per scheduler): warp 0 producer, 1 issuer, 2-17 epilogue
constexpr int GEMMF2_THREADS = 576;
__host__ __device__ constexpr int gemm2_threads(int epi) { return epi == 2 ? GEMMF2_THREADS : gemm_threads(epi); }
__host__ __device__ constexpr int epi_warps2(int epi) { return epi == 2 ? 16 : (epi == 3 ? 8 : 4); }
constexpr int GEMM_SMEM = STAGES * STAGE_BYTES + 1024;
constexpr int TMEM_COLS = 512;  // two accumulator buffers of up to 256 columns

enum { EPI_XPROJ = 0, EPI_LEVEL = 1, EPI_F = 2, EPI_XPROJ8 = 3 };
// EPI_XPROJ8 is the input projection with eight epilogue warps (used where the bf16 copy of h is kept in child order,
// i.e. ahead of per-level launches): its epilogue, like the forget-gate one, is bound by how many instructions one
// warp per scheduler can issue, so two warps per TMEM lane quarter share a tile's steps.
__host__ __device__ constexpr bool is_xproj(int epi) { return epi == EPI_XPROJ || epi == EPI_XPROJ8; }
__host__ __device__ constexpr int epi_warps(int epi) { return (epi == EPI_F || epi == EPI_XPROJ8) ? 8 : 4; }

struct TcArgs {
    const int32_t* child_ptr;
    const int32_t* child_idx;
    const int32_t* level_ptr;
    const int32_t* perm;
    int32_t* meta;
    int32_t n_nodes, n_edges, n_int_bound, H, Hp;
    const float* bias4;   // [Hp][4]
    float* P;             // [n_internal][4][Hp]   row = perm position - n_leaves, planes i, o, u, f
    float* S;             // [n_internal][Hp]      sum_k f_jk c_k, row = perm position - n_leaves (zeroed per call)
    __nv_bfloat16* hs;    // [n_internal][Hp]      child sums, row = perm position - n_leaves
    __nv_bfloat16* hb;    // [n_nodes][Hp]         bf16 copy of h: row = slot of the node as a child (child_order), or
                          //                       row = perm position (cooperative loop)
    float* h;
    float* c;
    int64_t ldh;
    int32_t vec_ok;       // h/c rows allow 16-byte accesses
    int32_t* inv;         // position of every node in level order
    int32_t p_tma;        // rows in level order (P; the bf16 copy of leaf rows when it is kept by position) leave
                          // through TMA stores
    int32_t issuers;      // MMA issuer warps of the lone-CTA GEMM: 1 (whole tile width) or 2 (half each)
    // the child-ordered layout of the per-level launches
    int32_t child_order;
    int32_t* eoff;        // [n_internal + 1]  first slot of every internal node's children, row = position - n_leaves
    int32_t* slot_of_pos; // [n_nodes]         slot of the node at a position in level order (-1: a root)
    int32_t* slot_par;    // [n_edges]         row (position - n_leaves) of the parent that owns the slot
    int32_t* slot_child;  // [n_edges]         node id of the child at the slot
    int32_t debug;        // check every index against its array before following it
    int32_t x_gather;     // the input projection reads its rows straight from the caller's x, picked by perm (TMA row gather)
};

// Where a tile sits.  The input projection walks the rows in level order and never mixes
// leaves and internal nodes in a tile: leaf tiles need only the i, o, u blocks (192 of the 256 columns of a
// 64-wide hidden slice), internal tiles all four.  The other GEMMs walk one contiguous range with a fixed N.
struct Tile {
    int n_tile, row0, row_end, bn;
};
template <int EPI>
__device__ __forceinline__ Tile tile_of(int t, int n_tiles, int tm, int lo, int hi, int bn, int n_leaves, int mt_leaf) {
    Tile r;
    const int m_tile = t / n_tiles;
    r.n_tile = t - m_tile * n_tiles;
    if (is_xproj(EPI)) {
        const bool leaf = m_tile < mt_leaf;
        r.row0 = leaf ? m_tile * tm : n_leaves + (m_tile - mt_leaf) * tm;
        r.row_end = leaf ? n_leaves : hi;
        r.bn = leaf ? 192 : 256;
    } else {
        r.row0 = lo + m_tile * tm;
        r.row_end = hi;
        r.bn = bn;
    }
    return r;
}


// ---- coalesced epilogue of a level tile ------------------------------------------------------------------
// An accumulator row lives in one thread (TMEM lane = row), but memory wants a warp's 16-byte pieces side by
// side: four lanes per row cover the 64 bytes a row contributes per 16-column step, eight rows per request.
// Each epilogue warp therefore owns a ring of three step buffers, each four [32 rows][16 floats] arrays, which
// cp.async fills with the P and S slices two steps ahead (across tile boundaries, so the first steps of a tile
// arrive while its main loop is still running) and through which c, h and the bf16 copy of h go out.
// A row's four 16-byte chunks are XOR-swizzled with bits 1..2 of the row, which keeps both the row-per-lane
// and the four-lanes-per-row accesses free of bank conflicts without padding.
constexpr int EPI_STEP_FLOATS = 4 * 32 * 16;              // one step buffer of one epilogue warp
constexpr int EPI_RING = 3;
constexpr int EPI_SCRATCH_BYTES = 4 * EPI_RING * EPI_STEP_FLOATS * 4;
constexpr int LEVEL_BN = 192;
constexpr int LEVEL_STAGES = 3;
constexpr int LEVEL_STAGE_BYTES = A_BYTES + LEVEL_BN * BK * 2;
constexpr int GEMM_SMEM_LEVEL = LEVEL_STAGES * LEVEL_STAGE_BYTES + EPI_SCRATCH_BYTES + 1024;
constexpr int GEMM_SMEM_STORE = GEMM_SMEM + 4 * EPI_STEP_FLOATS * 4;   // input projection: one step buffer per warp
// forget-gate GEMM: three full-width stages and a ring of three step buffers per warp, each two [32 rows][16 floats]
// arrays (the parent's forget pre-activation and the child's c)
constexpr int F_STEP_FLOATS = 2 * 32 * 16;
constexpr int F_STAGES = 3;
constexpr int F_WARPS = 8;
// A lone CTA: eight epilogue warps, each walking 128 of the tile's 256 edges.  A CTA of a pair holds half of B per
// stage, which leaves room for sixteen warps (64 edges each) with three pipeline stages.  Two step buffers per warp: the
// copies of a step start one step ahead (a third buffer, tried in the pair kernel, changed nothing).
__host__ __device__ constexpr int f_warps(bool pair) { return pair ? 16 : 8; }
__host__ __device__ constexpr int f_seg(bool pair) { return pair ? 64 : 128; }
__host__ __device__ constexpr int f_ring(bool pair) { return 2; }
constexpr int F_SCRATCH_BYTES = f_warps(false) * f_ring(false) * F_STEP_FLOATS * 4;
constexpr int F_SCRATCH2_BYTES = f_warps(true) * f_ring(true) * F_STEP_FLOATS * 4;
constexpr int STAGES2_F = 3;
constexpr int GEMM_SMEM_F = F_STAGES * STAGE_BYTES + F_SCRATCH_BYTES + 1024;
constexpr int X8_STAGES = 3;
constexpr int GEMM_SMEM_X8 = X8_STAGES * STAGE_BYTES + 8 * EPI_STEP_FLOATS * 4 + 1024;   // eight warps, one step buffer each
static_assert(GEMM_SMEM_X8 <= 227 * 1024 - 256, "GEMM shared memory");
static_assert(GEMM_SMEM_STORE <= 227 * 1024 - 256, "GEMM shared memory");
static_assert(GEMM_SMEM_F <= 227 * 1024 - 256, "forget GEMM shared memory");
static_assert(GEMM_SMEM_LEVEL <= 227 * 1024 - 256, "level GEMM shared memory");

__device__ __forceinline__ int sw_off(int row, int chunk) { return row * 16 + ((chunk ^ ((row >> 1) & 3)) << 2); }

__device__ __forceinline__ void cp_async16_zfill(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
// the same through L1 (rows that many lanes of the CTA ask for again and again: a parent's row, once per child)
__device__ __forceinline__ void cp_async16_ca_zfill(uint32_t dst, const void* src, uint32_t src_bytes) {
    asm volatile("cp.async.ca.shared.global [%0], [%1], 16, %2;" ::"r"(dst), "l"(src), "r"(src_bytes) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N>
__device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }

// Starts the copies of one step's P_i, P_o, P_u and S slices (rows past the range are zero-filled).
__device__ __forceinline__ void level_fetch(const TcArgs& a, const Tile& ti, int quarter, int lane, int q, int n_leaves,
                                            uint32_t buf) {
    const int col = ti.n_tile * 64 + q * 16 + (lane & 3) * 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = (lane >> 2) + 8 * i;
        const int p = ti.row0 + quarter * 32 + row;
        const bool valid = p < ti.row_end;
        const size_t r = valid ? (size_t)(p - n_leaves) : 0;
        const uint32_t nb = valid ? 16u : 0u;
        const float* prow = a.P + r * 4 * a.Hp + col;
        const uint32_t d = buf + (uint32_t)sw_off(row, lane & 3) * 4;
        cp_async16_zfill(d, prow, nb);
        cp_async16_zfill(d + 2048, prow + a.Hp, nb);
        cp_async16_zfill(d + 4096, prow + 2 * a.Hp, nb);
        cp_async16_zfill(d + 6144, a.S + r * a.Hp + col, nb);
    }
}

// Writes one step's c and h (fp32, rows by node id) and the bf16 copy of h (rows in level order) of this warp's
// 32 rows through the step buffer, so that four lanes cover a row's 64 bytes.
// HB_TILE: the bf16 copy is not stored here but collected, across the four steps of a tile, as a [32 rows][64 columns]
// tile in the second half of the step buffer (128-byte rows, 16-byte chunk c of row r at chunk c ^ (r & 7)), which the
// caller sends off as one TMA store.
// hbr: rows of the bf16 copy that receive tile rows (lane >> 1) and (lane >> 1) + 16 of this warp (-1: none), when
// the copy is stored here.
template <bool HB_TILE = false>
__device__ __forceinline__ void store_hc_step(const TcArgs& a, const Tile& ti, int quarter, int lane, int q, const int (&vs)[4],
                                              const int (&hbr)[2], const float (&cv)[16], const float (&hv)[16], float* sc) {
    const int lr = lane >> 2, lc = lane & 3;
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
        const int o = sw_off(lane, c4);
        *reinterpret_cast<float4*>(sc + o) = make_float4(cv[4 * c4], cv[4 * c4 + 1], cv[4 * c4 + 2], cv[4 * c4 + 3]);
        *reinterpret_cast<float4*>(sc + 512 + o) = make_float4(hv[4 * c4], hv[4 * c4 + 1], hv[4 * c4 + 2], hv[4 * c4 + 3]);
    }
    {
        uint32_t w[8];
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            __nv_bfloat162 p2 = __floats2bfloat162_rn(hv[2 * i], hv[2 * i + 1]);
            w[i] = *reinterpret_cast<uint32_t*>(&p2);
        }
        if (HB_TILE) {
            uint8_t* row = reinterpret_cast<uint8_t*>(sc) + 4096 + lane * 128;
            *reinterpret_cast<uint4*>(row + (((2 * q) ^ (lane & 7)) << 4)) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(row + (((2 * q + 1) ^ (lane & 7)) << 4)) = make_uint4(w[4], w[5], w[6], w[7]);
        } else {
            *reinterpret_cast<uint4*>(sc + 1024 + sw_off(lane, 0)) = make_uint4(w[0], w[1], w[2], w[3]);
            *reinterpret_cast<uint4*>(sc + 1024 + sw_off(lane, 1)) = make_uint4(w[4], w[5], w[6], w[7]);
        }
    }
    __syncwarp();
    const int j = ti.n_tile * 64 + q * 16 + lc * 4;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        if (vs[i] < 0) continue;
        const float4 cc = *reinterpret_cast<const float4*>(sc + sw_off(lr + 8 * i, lc));
        const float4 hh = *reinterpret_cast<const float4*>(sc + 512 + sw_off(lr + 8 * i, lc));
        float* cd = a.c + (int64_t)vs[i] * a.ldh + j;
        float* hd = a.h + (int64_t)vs[i] * a.ldh + j;
        if (a.vec_ok && j + 4 <= a.H) {
            *reinterpret_cast<float4*>(cd) = cc;
            *reinterpret_cast<float4*>(hd) = hh;
        } else {
            const float ce[4] = {cc.x, cc.y, cc.z, cc.w}, he[4] = {hh.x, hh.y, hh.z, hh.w};
#pragma unroll
            for (int e = 0; e < 4; ++e)
                if (j + e < a.H) { cd[e] = ce[e]; hd[e] = he[e]; }
        }
    }
    if (!HB_TILE) {
#pragma unroll
        for (int i = 0; i < 2; ++i) {  // bf16 copy of h: 32 bytes per row, two lanes per row
            const int r = (lane >> 1) + 16 * i;
            if (hbr[i] >= 0)
                *reinterpret_cast<uint4*>(a.hb + (size_t)hbr[i] * a.Hp + ti.n_tile * 64 + q * 16 + (lane & 1) * 8) =
                    *reinterpret_cast<const uint4*>(sc + 1024 + sw_off(r, lane & 1));
        }
    }
    __syncwarp();  // the arrays are free for the next step
}

// One 16-column step of a level tile for this warp's 32 rows: `sc` holds the step's P and S slices.
__device__ __forceinline__ void level_step(const TcArgs& a, const Tile& ti, uint32_t taddr, int quarter, int lane, int q,
                                           const int (&vs)[4], const int (&hbr)[2], float* sc) {
    float gi[16], go[16], gu[16];
    tmem_ld16(taddr + q * 16, gi);
    tmem_ld16(taddr + 64 + q * 16, go);
    tmem_ld16(taddr + 128 + q * 16, gu);
    tmem_ld_wait();
    float cv[16], hv[16];
#pragma unroll
    for (int c4 = 0; c4 < 4; ++c4) {
        const int o = sw_off(lane, c4);
        const float4 pi = *reinterpret_cast<const float4*>(sc + o), po = *reinterpret_cast<const float4*>(sc + 512 + o);
        const float4 pu = *reinterpret_cast<const float4*>(sc + 1024 + o), sv = *reinterpret_cast<const float4*>(sc + 1536 + o);
        cv[4 * c4 + 0] = fmaf(sigmoid_fast(gi[4 * c4 + 0] + pi.x), tanh_fast(gu[4 * c4 + 0] + pu.x), sv.x);
        cv[4 * c4 + 1] = fmaf(sigmoid_fast(gi[4 * c4 + 1] + pi.y), tanh_fast(gu[4 * c4 + 1] + pu.y), sv.y);
        cv[4 * c4 + 2] = fmaf(sigmoid_fast(gi[4 * c4 + 2] + pi.z), tanh_fast(gu[4 * c4 + 2] + pu.z), sv.z);
        cv[4 * c4 + 3] = fmaf(sigmoid_fast(gi[4 * c4 + 3] + pi.w), tanh_fast(gu[4 * c4 + 3] + pu.w), sv.w);
        hv[4 * c4 + 0] = sigmoid_fast(go[4 * c4 + 0] + po.x) * tanh_fast(cv[4 * c4 + 0]);
        hv[4 * c4 + 1] = sigmoid_fast(go[4 * c4 + 1] + po.y) * tanh_fast(cv[4 * c4 + 1]);
        hv[4 * c4 + 2] = sigmoid_fast(go[4 * c4 + 2] + po.z) * tanh_fast(cv[4 * c4 + 2]);
        hv[4 * c4 + 3] = sigmoid_fast(go[4 * c4 + 3] + po.w) * tanh_fast(cv[4 * c4 + 3]);
    }
    __syncwarp();  // every lane has read its inputs: the arrays now carry the outputs
    store_hc_step(a, ti, quarter, lane, q, vs, hbr, cv, hv, sc);
}

// x-projection step of a leaf tile: the cell finishes here (no children, so c = i u and h = o tanh(c)).
template <bool HB_TILE>
__device__ __forceinline__ void xproj_leaf_step(const TcArgs& a, const Tile& ti, uint32_t taddr, int quarter, int lane, int q,
                                                const int (&vs)[4], const int (&hbr)[2], float* sc) {
    const float4* bias4 = reinterpret_cast<const float4*>(a.bias4);
    float gi[16], go[16], gu[16];
    tmem_ld16(taddr + q * 16, gi);
    tmem_ld16(taddr + 64 + q * 16, go);
    tmem_ld16(taddr + 128 + q * 16, gu);
    tmem_ld_wait();
    const int j = ti.n_tile * 64 + q * 16;
    float cv[16], hv[16];
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float4 b = __ldg(&bias4[j + i]);
        const float cc = sigmoid_fast(gi[i] + b.x) * tanh_fast(gu[i] + b.z);
        cv[i] = cc;
        hv[i] = sigmoid_fast(go[i] + b.y) * tanh_fast(cc);
    }
    store_hc_step<HB_TILE>(a, ti, quarter, lane, q, vs, hbr, cv, hv, sc);
}

// x-projection step of a tile of internal nodes: the four biased pre-activations go to the planes of P.
__device__ __forceinline__ void xproj_internal_step(const TcArgs& a, const Tile& ti, uint32_t taddr, int quarter, int lane,
                                                    int q, int n_leaves, float* sc) {
    const float4* bias4 = reinterpret_cast<const float4*>(a.bias4);
    const int lr = lane >> 2, lc = lane & 3;
    float g[4][16];
#pragma unroll
    for (int k = 0; k < 4; ++k) tmem_ld16(taddr + k * 64 + q * 16, g[k]);
    tmem_ld_wait();
    const int j = ti.n_tile * 64 + q * 16;
#pragma unroll
    for (int i = 0; i < 16; ++i) {
        const float4 b = __ldg(&bias4[j + i]);
        g[0][i] += b.x; g[1][i] += b.y; g[2][i] += b.z; g[3][i] += b.w;
    }
#pragma unroll
    for (int k = 0; k < 4; ++k)
#pragma unroll
        for (int c4 = 0; c4 < 4; ++c4)
            *reinterpret_cast<float4*>(sc + k * 512 + sw_off(lane, c4)) =
                make_float4(g[k][4 * c4], g[k][4 * c4 + 1], g[k][4 * c4 + 2], g[k][4 * c4 + 3]);
    __syncwarp();
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int row = lr + 8 * i, p = ti.row0 + quarter * 32 + row;
        if (p >= ti.row_end) continue;
        float* prow = a.P + (size_t)(p - n_leaves) * 4 * a.Hp + j + lc * 4;
#pragma unroll
        for (int k = 0; k < 4; ++k)
            *reinterpret_cast<float4*>(prow + k * a.Hp) = *reinterpret_cast<const float4*>(sc + k * 512 + sw_off(row, lc));
    }
    __syncwarp();
}

// The same for a whole tile through the copy engine: P rows sit in level order, so a warp's 32 rows x 64 columns of one
// plane are a plain 2-D box.  Per plane the warp lays two [32 rows][32 floats] halves into its step buffer in the
// 128-byte swizzle of the tensor map (16-byte chunk c of row r at chunk c ^ (r & 7): one row per lane, conflict-free)
// and lane 0 sends them off as two TMA stores; the load/store units see the staging writes only.  Rows past the last
// internal node are dropped by the tensor map's bounds (or land in unused rows of P when its row count is a bound).
__device__ __forceinline__ void xproj_internal_tile_tma(const TcArgs& a, const Tile& ti, const CUtensorMap* tmP, uint32_t taddr,
                                                        int quarter, int lane, int n_leaves, float* sc, int k_begin, int k_end) {
    const float* bias = a.bias4;
    const int y = ti.row0 + quarter * 32 - n_leaves;
#pragma unroll 1
    for (int k = k_begin; k < k_end; ++k) {  // the planes (i, o, u, f) this warp sends off
        if (lane == 0) bulk_wait_read();  // the stores of the plane before have read the buffer
        __syncwarp();
#pragma unroll
        for (int half = 0; half < 2; ++half) {
            float g0[16], g1[16];
            tmem_ld16(taddr + k * 64 + half * 32, g0);
            tmem_ld16(taddr + k * 64 + half * 32 + 16, g1);
            tmem_ld_wait();
            const int j = ti.n_tile * 64 + half * 32;
            uint8_t* row = reinterpret_cast<uint8_t*>(sc) + half * 4096 + lane * 128;
#pragma unroll
            for (int c = 0; c < 8; ++c) {
                const float* g = c < 4 ? &g0[4 * c] : &g1[4 * (c - 4)];
                float4 v;
                v.x = g[0] + __ldg(&bias[4 * (j + 4 * c + 0) + k]);
                v.y = g[1] + __ldg(&bias[4 * (j + 4 * c + 1) + k]);
                v.z = g[2] + __ldg(&bias[4 * (j + 4 * c + 2) + k]);
                v.w = g[3] + __ldg(&bias[4 * (j + 4 * c + 3) + k]);
                *reinterpret_cast<float4*>(row + ((c ^ (lane & 7)) << 4)) = v;
            }
        }
        fence_proxy_async();  // this lane's rows are visible to the copy engine
        __syncwarp();
        if (lane == 0) {
            const int x = k * a.Hp + ti.n_tile * 64;
            tma_store_2d(tmP, smem_u32(sc), x, y);
            tma_store_2d(tmP, smem_u32(sc) + 4096, x + 32, y);
            bulk_commit();
        }
    }
    if (lane == 0) bulk_wait_read();  // the step buffer is free for whatever tile comes next
    __syncwarp();
}

// ---- epilogue of a forget-gate tile ---------------------------------------------------------------------------
// The accumulator holds (hidden unit, edge): TMEM lane = hidden unit, column = edge slot, 256 edges per tile, sorted by
// parent.  A warp owns 32 hidden units (its lane quarter) and a segment of 128 consecutive edges, walked in eight
// steps of 16 edges.  Per step it needs, for each edge, 32 floats of the parent's forget pre-activation P_f and of
// the child's c: [16 edges][32 floats] arrays in shared memory, filled by 16-byte asynchronous copies one step ahead
// (eight lanes per edge row) and read one float per lane, free of bank conflicts.
constexpr int F_EDGES = 256;      // edges per tile (the MMA's N)
// pr, kd: parent row and child node id of this lane's edges lane + 32 i of the segment, chosen for the step by the caller
__device__ __forceinline__ void forget_fetch(const TcArgs& a, int j_base, int lane, int st, int pr_sel, int kd_sel, uint32_t buf,
                                             float* bufp) {
    const int chunk = lane & 7, col = j_base + chunk * 4;
#pragma unroll
    for (int k = 0; k < 4; ++k) {
        const int er = (lane >> 3) + 4 * k;                       // edge row of the step
        const int src_lane = (st & 1) * 16 + er;                  // the lane that holds this edge's parent and child
        const int par = __shfl_sync(0xffffffffu, pr_sel, src_lane), kid = __shfl_sync(0xffffffffu, kd_sel, src_lane);
        const int o = er * 32 + chunk * 4;
        const uint32_t d = buf + (uint32_t)o * 4;
        const bool have = par >= 0 && col < a.Hp;
        cp_async16_ca_zfill(d, have ? a.P + ((size_t)par * 4 + 3) * a.Hp + col : a.P, have ? 16u : 0u);
        const int left = have ? a.H - col : 0;   // columns of the child's c row from `col` on
        if (left >= 4 && a.vec_ok) {
            cp_async16_zfill(d + 2048, a.c + (int64_t)kid * a.ldh + col, 16u);
        } else if (left <= 0) {
            cp_async16_zfill(d + 2048, a.P, 0u);
        } else {  // ragged end of the row, or rows that are not 16-byte aligned
            const float* src = a.c + (int64_t)kid * a.ldh + col;
            float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
            v.x = __ldcg(src);
            if (left > 1) v.y = __ldcg(src + 1);
            if (left > 2) v.z = __ldcg(src + 2);
            if (left > 3) v.w = __ldcg(src + 3);
            *reinterpret_cast<float4*>(bufp + 512 + o) = v;
        }
    }
}

// What a warp knows about its segment of a tile.
struct Segment {
    int pr[4], kd[4];        // parent row / child id of edges lane + 32 i (-1: no such edge)
    unsigned heads[4];       // bit e of word i: edge 32 i + e starts a new parent
    bool cont_before;        // the first parent's children start before this segment
    bool cont_after;         // the last parent's children go on behind this segment
};
__device__ __forceinline__ int sel4(const int (&v)[4], int i) { return i == 0 ? v[0] : i == 1 ? v[1] : i == 2 ? v[2] : v[3]; }
__device__ __forceinline__ unsigned sel4u(const unsigned (&v)[4], int i) { return i == 0 ? v[0] : i == 1 ? v[1] : i == 2 ? v[2] : v[3]; }

template <int SEG>
__device__ __forceinline__ Segment segment_of(const TcArgs& a, int slot0, int row_end, int lane) {
    constexpr int NI = SEG / 32;
    Segment sg;
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        const int sl = slot0 + 32 * i + lane;
        sg.pr[i] = sg.kd[i] = -1;
        sg.heads[i] = 0;
        if (i < NI && sl < row_end) {
            sg.pr[i] = a.slot_par[sl];
            sg.kd[i] = a.slot_child[sl];
            if (a.debug && (!dbg_ok(a.meta, CHECK_PARENT_ROW, sg.pr[i], a.n_int_bound, sl) ||
                            !dbg_ok(a.meta, CHECK_CHILD, sg.kd[i], a.n_nodes, sl)))
                sg.pr[i] = sg.kd[i] = -1;
        }
    }
#pragma unroll
    for (int i = 0; i < NI; ++i) {
        int prev = __shfl_up_sync(0xffffffffu, sg.pr[i], 1);
        const int carry = __shfl_sync(0xffffffffu, sg.pr[i > 0 ? i - 1 : 0], 31);
        if (lane == 0) prev = carry;
        sg.heads[i] = __ballot_sync(0xffffffffu, (i == 0 && lane == 0) || sg.pr[i] != prev);
    }
    const int n_valid = min(max(row_end - slot0, 0), SEG);
    const int p_first = __shfl_sync(0xffffffffu, sg.pr[0], 0);
    sg.cont_before = p_first >= 0 && a.eoff[p_first] != slot0;
    sg.cont_after = false;
    if (n_valid == SEG) {
        const int p_last = __shfl_sync(0xffffffffu, sg.pr[NI - 1], 31);
        sg.cont_after = p_last >= 0 && a.eoff[p_last + 1] != slot0 + SEG;
    }
    return sg;
}

// The running sum of one parent's f c_k in this thread's hidden unit, and where it goes when the parent's edges end:
// a plain store if all of the parent's edges lie in this segment, else an atomic addition (S starts at zero; a parent
// whose children straddle segments receives one contribution from each).
struct RunSum {
    float sum;
    int par, runs_done;
};
__device__ __forceinline__ void run_flush(float* S, int Hp, float sum, int par, int j, bool j_ok, bool partial) {
    if (par < 0 || !j_ok) return;
    float* dst = S + (size_t)par * Hp + j;
    if (partial) asm volatile("red.global.add.f32 [%0], %1;" ::"l"(dst), "f"(sum) : "memory");
    else *dst = sum;
}

// One step of 16 edges for this thread's hidden unit.
__device__ __forceinline__ void forget_step(const TcArgs& a, const Segment& sg, uint32_t taddr, int lane, int st, int j, bool j_ok,
                                            RunSum& r, const float* sc) {
    float g[16];
    tmem_ld16(taddr + st * 16, g);
    tmem_ld_wait();
    const unsigned heads = sel4u(sg.heads, st >> 1) >> ((st & 1) * 16);
    const int pr_sel = sel4(sg.pr, st >> 1);
    // first all sixteen products, free of branches, so that their chains of dependent instructions (shared-memory
    // load, add, tanh, multiply) overlap; then the cheap serial part, which alone depends on where parents change
    float fc[16];
#pragma unroll
    for (int e = 0; e < 16; ++e) fc[e] = sigmoid_fast(sc[e * 32 + lane] + g[e]) * sc[512 + e * 32 + lane];
#pragma unroll
    for (int e = 0; e < 16; ++e) {
        if ((heads >> e) & 1u) {   // the same in every lane: a new parent starts at this edge
            run_flush(a.S, a.Hp, r.sum, r.par, j, j_ok, r.runs_done == 0 && sg.cont_before);
            r.par = __shfl_sync(0xffffffffu, pr_sel, (st & 1) * 16 + e);
            r.sum = 0.f;
            ++r.runs_done;
        }
        r.sum += fc[e];
    }
}

// The epilogue warps of a GEMM CTA (the four warps whose index modulo 4 selects a TMEM lane quarter): for every
// tile of this CTA, wait for the accumulator, run the fused arithmetic and stores, hand the accumulator back.
// PAIR: the CTA is one of a cta_group::2 pair working on a 256-row tile; it owns rows rank*128.. of the tile,
// waits on its own copy of the accumulator barrier and releases the accumulator at the pair leader.
// `scratch` is this CTA's epilogue shared memory (ring or step buffers of the four warps).
template <int EPI, bool PAIR>
__device__ __forceinline__ void epilogue_warps(const TcArgs& a, const CUtensorMap* tmP, const CUtensorMap* tmHB,
                                               float* scratch, uint32_t tmem_base, uint64_t* bar_tfull,
                                               uint64_t* bar_tempty, volatile int* abort, int warp, int lane, int t0, int t_step,
                                               int total_tiles, int n_tiles, int lo, int hi, int bn, int n_leaves, int mt_leaf,
                                               int rank) {
    constexpr int TM = PAIR ? 2 * BM : BM;
    auto tile_at = [&](int t) {   // (not for the forget-gate GEMM, whose tiles are laid out differently)
        Tile ti = tile_of<EPI>(t, n_tiles, TM, lo, hi, bn, n_leaves, mt_leaf);
        if (PAIR) ti.row0 += rank * BM;
        return ti;
    };
    // the verdict is taken over the whole warp: the accumulator loads that follow are warp-wide instructions
    auto wait_acc = [&](int acc, uint32_t phase) {
        const bool mine = PAIR ? mbar_wait_cluster(smem_u32(&bar_tfull[acc]), phase, abort) : mbar_wait(smem_u32(&bar_tfull[acc]), phase, abort);
        return __all_sync(0xffffffffu, mine) != 0;
    };
    auto release_acc = [&](int acc) {
        tc_fence_before();
        if (PAIR) mbar_arrive_cluster(mapa_u32(smem_u32(&bar_tempty[acc]), 0));
        else mbar_arrive(smem_u32(&bar_tempty[acc]));
    };
    const int quarter = warp & 3;           // TMEM lane quarter this warp may read
    // node id of the row at position p (rows this lane stores), and the row of the bf16 copy that receives it
    auto node_at = [&](int p, int row_end) {
        if (p >= row_end) return -1;
        const int v = a.perm[p];
        if (a.debug && !dbg_ok(a.meta, CHECK_PERM, v, a.n_nodes, p)) return -1;
        return v;
    };
    auto copy_row_at = [&](int p, int row_end) {
        if (p >= row_end) return -1;
        if (!a.child_order) return p;
        const int sl = a.slot_of_pos[p];
        if (a.debug && sl >= 0 && !dbg_ok(a.meta, CHECK_SLOT, sl, a.n_edges, p)) return -1;
        return sl;
    };
    int acc = 0;
    uint32_t acc_phase = 0;
    bool ok = true;
    if (EPI == EPI_LEVEL) {
        // coalesced epilogue; the copies of a step's P and S slices run two steps ahead of its arithmetic
        float* ring = scratch + quarter * (EPI_RING * EPI_STEP_FLOATS);
        const uint32_t ring_addr = smem_u32(ring);
        int f_t = t0, f_q = 0, f_buf = 0;  // the step whose copies start next
        Tile f_ti = tile_at(f_t);
        auto fetch_next = [&]() {
            if (f_t < total_tiles) {
                level_fetch(a, f_ti, quarter, lane, f_q, n_leaves, ring_addr + (uint32_t)f_buf * (EPI_STEP_FLOATS * 4));
                if (++f_q == 4) {
                    f_q = 0;
                    f_t += t_step;
                    f_ti = tile_at(f_t);
                }
            }
            cp_async_commit();  // one group per step, empty past the last tile
            if (++f_buf == EPI_RING) f_buf = 0;
        };
        fetch_next();
        fetch_next();
        int cur = 0;
        for (int t = t0; t < total_tiles && ok; t += t_step) {
            const Tile ti = tile_at(t);
            int vs[4], hbr[2];  // node ids of the rows this lane stores; rows of the bf16 copy
#pragma unroll
            for (int i = 0; i < 4; ++i) vs[i] = node_at(ti.row0 + quarter * 32 + (lane >> 2) + 8 * i, ti.row_end);
#pragma unroll
            for (int i = 0; i < 2; ++i) hbr[i] = copy_row_at(ti.row0 + quarter * 32 + (lane >> 1) + 16 * i, ti.row_end);
            if (!wait_acc(acc, acc_phase)) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + (uint32_t)acc * MAX_BN + ((uint32_t)(quarter * 32) << 16);
#pragma unroll 1
            for (int q = 0; q < 4; ++q) {
                fetch_next();                // into the buffer the previous step has just released
                cp_async_wait<2>();          // this step's own copies have landed
                __syncwarp();                // ... and so have the other lanes'
                level_step(a, ti, taddr, quarter, lane, q, vs, hbr, ring + cur * EPI_STEP_FLOATS);
                if (++cur == EPI_RING) cur = 0;
            }
            release_acc(acc);
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1u;
        }
        cp_async_wait<0>();
    } else if (EPI == EPI_F) {
        // eight or sixteen warps: lane quarter = 32 hidden units, segment = 128 or 64 consecutive edges of the tile
        constexpr int RING = f_ring(PAIR), F_SEG = f_seg(PAIR), STEPS = F_SEG / 16;
        const int seg = (warp - 2) >> 2;
        float* ring = scratch + (warp - 2) * (RING * F_STEP_FLOATS);
        const uint32_t ring_addr = smem_u32(ring);
        constexpr int TMH = PAIR ? 2 * BM : BM;   // hidden units per tile
        for (int t = t0; t < total_tiles && ok; t += t_step) {
            const Tile ti = tile_of<EPI>(t, n_tiles, F_EDGES, lo, hi, bn, n_leaves, mt_leaf);
            const int j_base = ti.n_tile * TMH + rank * BM + quarter * 32, j = j_base + lane;
            const bool j_ok = j < a.Hp;
            const int slot0 = ti.row0 + seg * F_SEG;
            const Segment sg = segment_of<F_SEG>(a, slot0, ti.row_end, lane);
            // the first steps' copies start before the accumulator is ready: they land while the tile's products run
#pragma unroll
            for (int st = 0; st < RING - 1; ++st) {
                forget_fetch(a, j_base, lane, st, sel4(sg.pr, st >> 1), sel4(sg.kd, st >> 1), ring_addr + (uint32_t)st * (F_STEP_FLOATS * 4),
                             ring + st * F_STEP_FLOATS);
                cp_async_commit();
            }
            if (!wait_acc(acc, acc_phase)) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + (uint32_t)acc * MAX_BN + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(seg * F_SEG);
            RunSum r{0.f, -1, -1};   // the first edge of the segment always starts a run: runs_done becomes 0 there
            int cur = 0, nxt = RING - 1;   // buffer of this step, buffer the next copies go to
#pragma unroll 1
            for (int st = 0; st < STEPS; ++st) {
                cp_async_wait<RING - 2>();   // this step's copies have landed (they were started RING - 1 steps ago)
                __syncwarp();                // ... and so have the other lanes'; the buffer of the step before is free
                if (st + RING - 1 < STEPS) {
                    const int sn = st + RING - 1;
                    forget_fetch(a, j_base, lane, sn, sel4(sg.pr, sn >> 1), sel4(sg.kd, sn >> 1),
                                 ring_addr + (uint32_t)nxt * (F_STEP_FLOATS * 4), ring + nxt * F_STEP_FLOATS);
                }
                cp_async_commit();
                forget_step(a, sg, taddr, lane, st, j, j_ok, r, ring + cur * F_STEP_FLOATS);
                if (++cur == RING) cur = 0;
                if (++nxt == RING) nxt = 0;
            }
            run_flush(a.S, a.Hp, r.sum, r.par, j, j_ok, (r.runs_done == 0 && sg.cont_before) || sg.cont_after);
            cp_async_wait<0>();
            __syncwarp();                    // every lane is done with the buffers before the next tile refills them
            release_acc(acc);
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1u;
        }
        cp_async_wait<0>();
    } else {
        // input projection: stores only; every step goes through one step buffer per warp to leave in coalesced pieces.
        // With eight warps the two warps of a lane quarter take the steps (or the planes of P) alternately.
        constexpr int NSPLIT = epi_warps(EPI) / 4;
        const int split = (warp - 2) >> 2;
        float* sc = scratch + (warp - 2) * EPI_STEP_FLOATS;
        for (int t = t0; t < total_tiles && ok; t += t_step) {
            const Tile ti = tile_at(t);
            const bool leaf = ti.bn == 192;
            // node ids, fetched while the main loop of this tile is still running
            int vs[4], hbr[2];
#pragma unroll
            for (int i = 0; i < 4; ++i) vs[i] = leaf ? node_at(ti.row0 + quarter * 32 + (lane >> 2) + 8 * i, ti.row_end) : -1;
#pragma unroll
            for (int i = 0; i < 2; ++i) hbr[i] = leaf ? copy_row_at(ti.row0 + quarter * 32 + (lane >> 1) + 16 * i, ti.row_end) : -1;
            if (!wait_acc(acc, acc_phase)) { ok = false; break; }
            tc_fence_after();
            const uint32_t taddr = tmem_base + (uint32_t)acc * MAX_BN + ((uint32_t)(quarter * 32) << 16);
            if (leaf) {
                if (NSPLIT == 1 && a.p_tma && !a.child_order) {
                    // the bf16 copy is kept by position: the tile's rows leave as one TMA store (a plain box).
                    // Rows of a partly filled last leaf tile belong to internal nodes, whose rows are written
                    // again, with their values, by the level that evaluates them.
                    if (lane == 0) bulk_wait_read();  // the store of the tile before has read the tile buffer
                    __syncwarp();
#pragma unroll 1
                    for (int q = 0; q < 4; ++q) xproj_leaf_step<true>(a, ti, taddr, quarter, lane, q, vs, hbr, sc);
                    fence_proxy_async();
                    __syncwarp();
                    if (lane == 0) {
                        tma_store_2d(tmHB, smem_u32(sc) + 4096, ti.n_tile * 64, ti.row0 + quarter * 32);
                        bulk_commit();
                    }
                } else {
#pragma unroll 1
                    for (int q = split; q < 4; q += NSPLIT) xproj_leaf_step<false>(a, ti, taddr, quarter, lane, q, vs, hbr, sc);
                }
            } else {
                if (a.p_tma) {
                    xproj_internal_tile_tma(a, ti, tmP, taddr, quarter, lane, n_leaves, sc, split * (4 / NSPLIT), (split + 1) * (4 / NSPLIT));
                } else {
#pragma unroll 1
                    for (int q = split; q < 4; q += NSPLIT) xproj_internal_step(a, ti, taddr, quarter, lane, q, n_leaves, sc);
                }
            }
            release_acc(acc);
            acc ^= 1;
            if (acc == 0) acc_phase ^= 1u;
        }
        if (lane == 0) bulk_wait_all();  // no store of this warp is still on its way
    }
    if (!ok) *abort = 1;
}

// Row range of one level's launch: positions of the level's nodes (gate GEMM), or the slots of their children
// (forget-gate GEMM).  An inconsistent range is recorded (debug checks) and made empty.
template <int EPI>
__device__ __forceinline__ void level_range(const TcArgs& a, int level, int n_leaves, int& lo, int& hi) {
    checked_level(a.level_ptr, level, a.n_nodes, a.meta, a.debug, lo, hi);
    bool good = !a.debug || (dbg_ok(a.meta, CHECK_LEVEL_PTR, lo - n_leaves, (long long)a.n_int_bound + 1, level) &&
                             dbg_ok(a.meta, CHECK_LEVEL_PTR, hi - n_leaves, (long long)a.n_int_bound + 1, level));
    if (good && EPI == EPI_F) {
        lo = a.eoff[lo - n_leaves];
        hi = a.eoff[hi - n_leaves];
        good = !a.debug || (dbg_ok(a.meta, CHECK_EDGE_PTR, lo, (long long)a.n_edges + 1, level) &&
                            dbg_ok(a.meta, CHECK_EDGE_PTR, hi, (long long)a.n_edges + 1, level) &&
                            dbg_ok(a.meta, CHECK_EDGE_PTR, hi - lo, (long long)a.n_edges + 1, level));
    }
    if (!good) lo = hi = 0;
}

template <int EPI>
__global__ void __launch_bounds__(gemm_threads(EPI), 1)
gemm_tc_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
               const __grid_constant__ CUtensorMap tmB_leaf, const __grid_constant__ CUtensorMap tmP,
               const __grid_constant__ CUtensorMap tmHBs, TcArgs a, int level, int bn, int n_total, int kblocks) {
    // the per-level GEMMs trade one pipeline stage (their K is the hidden size: few blocks) for the epilogue's ring
    constexpr int NST = EPI == EPI_LEVEL ? LEVEL_STAGES : EPI == EPI_F ? F_STAGES : EPI == EPI_XPROJ8 ? X8_STAGES : STAGES;
    constexpr int SB = EPI == EPI_LEVEL ? LEVEL_STAGE_BYTES : STAGE_BYTES;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[NST], bar_empty[NST], bar_tfull[2], bar_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < NST; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), a.issuers);  // one commit from each MMA issuer
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_tfull[b]), a.issuers);
            mbar_init(smem_u32(&bar_tempty[b]), 32 * epi_warps(EPI));
        }
        fence_barrier_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) tmem_alloc(smem_u32(&s_tmem_base), TMEM_COLS);
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort = &s_abort;

    // everything above touches no global memory; what follows reads what earlier kernels of the stream wrote
    griddep_wait();
    griddep_launch();

    // tile range of this launch (a level past the last one has no tiles: every role falls through to the end)
    int lo = 0, hi = 0, a_row_off = 0;
    const int n_levels = a.meta[META_N_LEVELS];
    const int n_leaves = n_levels > 0 ? a.level_ptr[1] : 0;
    if (is_xproj(EPI)) {
        hi = a.n_nodes;
    } else if (level < n_levels) {
        level_range<EPI>(a, level, n_leaves, lo, hi);
        a_row_off = (EPI == EPI_LEVEL) ? -n_leaves : 0;
    }
    const int mt_leaf = is_xproj(EPI) ? (n_leaves + BM - 1) / BM : 0;
    // forget-gate GEMM: tiles of 256 edges x 128 hidden units, the hidden tiles of an edge tile next to each other
    const int m_tiles = is_xproj(EPI) ? mt_leaf + (hi - n_leaves + BM - 1) / BM
                        : EPI == EPI_F ? (hi - lo + F_EDGES - 1) / F_EDGES : (hi - lo + BM - 1) / BM;
    const int n_tiles = EPI == EPI_F ? (a.Hp + BM - 1) / BM : n_total / bn;
    const int total_tiles = m_tiles * n_tiles;
    constexpr int TILE_ROWS = EPI == EPI_F ? F_EDGES : BM;

    if (warp == 0) {
        // producer warp: lane 0 waits for the stage and issues the tile loads.  With x_gather the rows of the input
        // projection's A tile are rows of the caller's x picked by perm: every lane holds four of the tile's node ids
        // and issues one four-row gather per K block (rows past the tile's end repeat its last row; nobody reads them).
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        const bool gather = is_xproj(EPI) && a.x_gather;
        for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
            const Tile ti = tile_of<EPI>(t, n_tiles, TILE_ROWS, lo, hi, bn, n_leaves, mt_leaf);
            const uint32_t tx = A_BYTES + (uint32_t)ti.bn * BK * 2;
            int rows[4] = {0, 0, 0, 0};
            if (gather) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int p = min(ti.row0 + 4 * lane + i, ti.row_end - 1);
                    int v = a.perm[p];
                    if (a.debug && !dbg_ok(a.meta, CHECK_PERM, v, a.n_nodes, p)) v = 0;
                    rows[i] = v;
                }
            }
            for (int kb = 0; kb < kblocks; ++kb) {
                const uint32_t full = smem_u32(&bar_full[stage]);
                if (lane == 0) {
                    ok = mbar_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, abort);
                    if (ok) {
                        mbar_expect_tx(full, tx);
                        // forget-gate GEMM: A = 128 rows (hidden units) of U_f, B = the tile's 256 edge rows of the bf16 copy
                        if (!gather) tma_load_2d(smem_base + stage * SB, &tmA, full, kb * BK, EPI == EPI_F ? ti.n_tile * BM : ti.row0 + a_row_off);
                        tma_load_2d(smem_base + stage * SB + A_BYTES, (is_xproj(EPI) && ti.bn == 192) ? &tmB_leaf : &tmB,
                                    full, kb * BK, is_xproj(EPI) ? ti.n_tile * 256 : EPI == EPI_F ? ti.row0 : ti.n_tile * bn);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                if (gather) tma_gather4_2d(smem_base + stage * SB + lane * 512, &tmA, full, kb * BK, rows[0], rows[1], rows[2], rows[3]);
                if (++stage == NST) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && lane == 0) *abort = 1;
    } else if (warp == 1 || (epi_warps(EPI) == 4 && warp == 6 && a.issuers == 2)) {
        // One MMA issuer for the whole tile width, or two taking half of the columns each.  The whole warp walks the pipeline (waits,
        // descriptors), so every operand of tcgen05.mma is warp-uniform; one elected lane issues.
        {
            const int half = warp == 6;
            const bool issuer = elect_one();
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int t = blockIdx.x; t < total_tiles && ok; t += gridDim.x) {
                const Tile ti = tile_of<EPI>(t, n_tiles, TILE_ROWS, lo, hi, bn, n_leaves, mt_leaf);
                const int hn = a.issuers == 2 ? ti.bn >> 1 : ti.bn;  // columns of this issuer
                const uint32_t idesc = idesc_bf16(BM, hn);
                ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_tempty[acc]), acc_phase ^ 1u, abort));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * MAX_BN + (uint32_t)(half * hn);
                for (int kb = 0; kb < kblocks; ++kb) {
                    ok = __all_sync(0xffffffffu, mbar_wait(smem_u32(&bar_full[stage]), phase, abort));
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t adesc = smem_desc_sw128(smem_base + stage * SB);
                    const uint64_t bdesc = smem_desc_sw128(smem_base + stage * SB + A_BYTES + half * hn * 128);
                    if (issuer) {
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            mma_bf16(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                        mma_commit(smem_u32(&bar_empty[stage]));
                    }
                    __syncwarp();
                    if (++stage == NST) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (issuer) mma_commit(smem_u32(&bar_tfull[acc]));
                __syncwarp();
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1u;
            }
            if (!ok && lane == 0) *abort = 1;
        }
    } else if (warp >= 2 && warp <= 1 + epi_warps(EPI)) {
        epilogue_warps<EPI, false>(a, &tmP, &tmHBs, reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)) + NST * SB), tmem_base,
                                   bar_tfull, bar_tempty, abort, warp, lane, blockIdx.x, gridDim.x, total_tiles, n_tiles, lo, hi,
                                   bn, n_leaves, mt_leaf, 0);
    }

    __syncthreads();
    if (s_abort) {
        // a bounded wait ran out: let copies that are still in flight land before the CTA's memory goes away
        if (threadIdx.x == 0) atomicExch(&a.meta[META_TIMEOUT], 1);
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
    tc_fence_after();
    if (warp == 1) tmem_dealloc(tmem_base, TMEM_COLS);
}

// The same pipeline over a PAIR of CTAs (cluster of 2, tcgen05 cta_group::2): the pair computes a 256-row tile,
// each CTA loads its own 128 rows of A and HALF of the B tile, and the leader's MMA reads both halves, so every SM
// pulls a third fewer operand bytes per flop from L2 than a lone CTA does (the single-CTA kernel is bound by the
// bytes it can keep in flight).  Barriers: the leader's `full` barrier collects the bytes of all four loads
// of a stage; `empty` and `tfull` are signalled in both CTAs by one multicast commit; the epilogue threads of
// both CTAs arrive on the leader's `tempty`.  Accumulator rows of CTA r are rows r*128.. of the tile.
constexpr int STAGES2 = 6, STAGES2_LEVEL = 4;
constexpr int STAGE2_BYTES = A_BYTES + B_BYTES_MAX / 2;
constexpr int GEMM2_SMEM = STAGES2 * STAGE2_BYTES + 4 * EPI_STEP_FLOATS * 4 + 1024;
constexpr int GEMM2_SMEM_LEVEL = STAGES2_LEVEL * STAGE2_BYTES + EPI_SCRATCH_BYTES + 1024;
constexpr int GEMM2_SMEM_F = STAGES2_F * STAGE2_BYTES + F_SCRATCH2_BYTES + 1024;
static_assert(GEMM2_SMEM_F <= 227 * 1024 - 256, "pair forget GEMM shared memory");
constexpr int GEMM2_SMEM_X8 = STAGES2_LEVEL * STAGE2_BYTES + 8 * EPI_STEP_FLOATS * 4 + 1024;
static_assert(GEMM2_SMEM_LEVEL <= 227 * 1024 - 256, "pair level GEMM shared memory");

template <int EPI>
__global__ void __launch_bounds__(gemm2_threads(EPI), 1)
gemm_tc2_kernel(const __grid_constant__ CUtensorMap tmA, const __grid_constant__ CUtensorMap tmB,
                const __grid_constant__ CUtensorMap tmB_leaf, const __grid_constant__ CUtensorMap tmP,
               const __grid_constant__ CUtensorMap tmHBs, TcArgs a, int level, int bn, int n_total, int kblocks) {
    // the kernels with rings or eight step buffers give up two stages, the sixteen-warp forget-gate kernel three
    constexpr int NST2 = EPI == EPI_XPROJ ? STAGES2 : EPI == EPI_F ? STAGES2_F : STAGES2_LEVEL;
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_full[NST2], bar_empty[NST2], bar_tfull[2], bar_tempty[2];
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort;

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t smem_base = (smem_u32(smem_raw) + 1023u) & ~1023u;
    const uint32_t rank = cluster_ctarank();
    const int pair = blockIdx.x >> 1, n_pairs = gridDim.x >> 1;

    griddep_wait();
    griddep_launch();
    int lo, hi, a_row_off;
    const int n_levels = a.meta[META_N_LEVELS];
    const int n_leaves = n_levels > 0 ? a.level_ptr[1] : 0;
    if (is_xproj(EPI)) {
        lo = 0; hi = a.n_nodes; a_row_off = 0;
    } else {
        if (level >= n_levels) return;  // uniform over the whole grid; nothing allocated, no cluster barrier yet
        level_range<EPI>(a, level, n_leaves, lo, hi);
        a_row_off = (EPI == EPI_LEVEL) ? -n_leaves : 0;
    }
    constexpr int TM2 = 2 * BM;
    const int mt_leaf = is_xproj(EPI) ? (n_leaves + TM2 - 1) / TM2 : 0;
    // forget-gate GEMM: tiles of 256 edges x 256 hidden units (128 per CTA)
    const int m_tiles = is_xproj(EPI) ? mt_leaf + (hi - n_leaves + TM2 - 1) / TM2 : (hi - lo + TM2 - 1) / TM2;
    const int n_tiles = EPI == EPI_F ? (a.Hp + TM2 - 1) / TM2 : n_total / bn;
    const int total_tiles = m_tiles * n_tiles;

    if (threadIdx.x == 0) {
        s_abort = 0;
        for (int s = 0; s < NST2; ++s) {
            mbar_init(smem_u32(&bar_full[s]), 1);
            mbar_init(smem_u32(&bar_empty[s]), 1);  // one multicast commit of the MMA issuer
        }
        for (int b = 0; b < 2; ++b) {
            mbar_init(smem_u32(&bar_tfull[b]), 1);
            mbar_init(smem_u32(&bar_tempty[b]), 64 * epi_warps2(EPI));  // the epilogue threads of both CTAs
        }
        fence_barrier_init();
        prefetch_tmap(&tmA);
        prefetch_tmap(&tmB);
    }
    if (warp == 1) tmem_alloc<2>(smem_u32(&s_tmem_base), TMEM_COLS);  // one warp of each CTA of the pair, together
    tc_fence_before();
    __syncthreads();
    cluster_sync();  // the peer's barriers exist before anything is sent to them
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort = &s_abort;

    if (warp == 0) {
        int stage = 0;
        uint32_t phase = 0;
        bool ok = true;
        const bool gather = is_xproj(EPI) && a.x_gather;
        for (int t = pair; t < total_tiles && ok; t += n_pairs) {
            const Tile ti = tile_of<EPI>(t, n_tiles, TM2, lo, hi, bn, n_leaves, mt_leaf);
            const int half_bn = ti.bn >> 1;
            const uint32_t tx = 2u * (A_BYTES + (uint32_t)half_bn * BK * 2);
            const int my_row0 = ti.row0 + (int)rank * BM;
            int rows[4] = {0, 0, 0, 0};   // x_gather: node ids of the four rows this lane fetches (see the lone-CTA kernel)
            if (gather) {
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const int p = min(my_row0 + 4 * lane + i, ti.row_end - 1);
                    int v = a.perm[p];
                    if (a.debug && !dbg_ok(a.meta, CHECK_PERM, v, a.n_nodes, p)) v = 0;
                    rows[i] = v;
                }
            }
            for (int kb = 0; kb < kblocks; ++kb) {
                const uint32_t full_leader = mapa_u32(smem_u32(&bar_full[stage]), 0);
                if (lane == 0) {
                    ok = mbar_wait(smem_u32(&bar_empty[stage]), phase ^ 1u, abort);
                    if (ok) {
                        if (rank == 0) mbar_expect_tx(smem_u32(&bar_full[stage]), tx);
                        // forget-gate GEMM: A = this CTA's 128 of the tile's 256 hidden units of U_f, B = its half of the edges
                        if (!gather) tma_load_2d_pair(smem_base + stage * STAGE2_BYTES, &tmA, full_leader, kb * BK,
                                                      EPI == EPI_F ? ti.n_tile * TM2 + (int)rank * BM : my_row0 + a_row_off);
                        // this CTA's half of the B tile's rows (the MMA reads rows 0.. from CTA 0, the rest from CTA 1)
                        const int n_base = is_xproj(EPI) ? ti.n_tile * 256 : EPI == EPI_F ? ti.row0 : ti.n_tile * bn;
                        const CUtensorMap* tb = (is_xproj(EPI) && ti.bn == 192) ? &tmB_leaf : &tmB;
                        tma_load_2d_pair(smem_base + stage * STAGE2_BYTES + A_BYTES, tb, full_leader, kb * BK,
                                         n_base + (int)rank * half_bn);
                    }
                }
                ok = __shfl_sync(0xffffffffu, ok ? 1 : 0, 0) != 0;
                if (!ok) break;
                if (gather) tma_gather4_2d_pair(smem_base + stage * STAGE2_BYTES + lane * 512, &tmA, full_leader, kb * BK, rows[0], rows[1], rows[2], rows[3]);
                if (++stage == NST2) { stage = 0; phase ^= 1u; }
            }
        }
        if (!ok && lane == 0) *abort = 1;
    } else if (warp == 1) {
        // the MMA issuer, in the leader CTA: the whole warp walks the pipeline so that every operand of tcgen05.mma
        // is warp-uniform; one elected lane issues
        if (rank == 0) {
            const bool issuer = elect_one();
            int stage = 0, acc = 0;
            uint32_t phase = 0, acc_phase = 0;
            bool ok = true;
            for (int t = pair; t < total_tiles && ok; t += n_pairs) {
                const Tile ti = tile_of<EPI>(t, n_tiles, TM2, lo, hi, bn, n_leaves, mt_leaf);
                const uint32_t idesc = idesc_bf16(2 * BM, ti.bn);
                ok = __all_sync(0xffffffffu, mbar_wait_cluster(smem_u32(&bar_tempty[acc]), acc_phase ^ 1u, abort));
                if (!ok) break;
                tc_fence_after();
                const uint32_t d_tmem = tmem_base + (uint32_t)acc * MAX_BN;
                for (int kb = 0; kb < kblocks; ++kb) {
                    ok = __all_sync(0xffffffffu, mbar_wait_cluster(smem_u32(&bar_full[stage]), phase, abort));
                    if (!ok) break;
                    tc_fence_after();
                    const uint64_t adesc = smem_desc_sw128(smem_base + stage * STAGE2_BYTES);
                    const uint64_t bdesc = smem_desc_sw128(smem_base + stage * STAGE2_BYTES + A_BYTES);
                    if (issuer) {
#pragma unroll
                        for (int k = 0; k < BK / 16; ++k)
                            mma_bf16_pair(d_tmem, adesc + 2 * k, bdesc + 2 * k, idesc, (kb | k) != 0 ? 1u : 0u);
                        mma_commit_pair(smem_u32(&bar_empty[stage]));
                    }
                    __syncwarp();
                    if (++stage == NST2) { stage = 0; phase ^= 1u; }
                }
                if (!ok) break;
                if (issuer) mma_commit_pair(smem_u32(&bar_tfull[acc]));
                __syncwarp();
                acc ^= 1;
                if (acc == 0) acc_phase ^= 1u;
            }
            if (!ok && lane == 0) *abort = 1;
        }
    } else if (warp >= 2 && warp <= 1 + epi_warps2(EPI)) {
        epilogue_warps<EPI, true>(a, &tmP, &tmHBs, reinterpret_cast<float*>(smem_raw + (smem_base - smem_u32(smem_raw)) + NST2 * STAGE2_BYTES),
                                  tmem_base, bar_tfull, bar_tempty, abort, warp, lane, pair, n_pairs, total_tiles, n_tiles, lo, hi,
                                  bn, n_leaves, mt_leaf, (int)rank);
    }

    __syncthreads();
    if (s_abort) {
        if (threadIdx.x == 0) atomicExch(&a.meta[META_TIMEOUT], 1);
        for (int i = 0; i < 200; ++i) __nanosleep(1000);
        __syncthreads();
    }
    cluster_sync();  // nothing of the peer (commits, arrivals) is still on its way to this CTA's memory
    tc_fence_after();
    if (warp == 1) tmem_dealloc<2>(tmem_base, TMEM_COLS);
}

// The operand of a level's gate GEMM, one warp per node: h~_j = sum_k bf16(h_k), fp32 adds in child-list order,
// rounded to bf16 once.  The child rows of a node are consecutive rows of the child-ordered copy, and the nodes of a
// level own consecutive runs of them, so the kernel streams one contiguous range with 16-byte loads.
__global__ void __launch_bounds__(256, 4) childsum_kernel(TcArgs a, int level) {
    griddep_wait();
    griddep_launch();
    const int n_levels = a.meta[META_N_LEVELS];
    if (level >= n_levels) return;
    const int n_leaves = a.level_ptr[1];
    int lo, hi;
    level_range<EPI_LEVEL>(a, level, n_leaves, lo, hi);
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    const int pieces = a.Hp >> 3;  // 16-byte pieces of a row
    for (int pos = lo + ((blockIdx.x * blockDim.x + threadIdx.x) >> 5); pos < hi; pos += warps) {
        const size_t r = (size_t)(pos - n_leaves);
        int e0 = a.eoff[r], e1 = a.eoff[r + 1];
        if (a.debug && (!dbg_ok(a.meta, CHECK_EDGE_PTR, e0, (long long)a.n_edges + 1, pos) ||
                        !dbg_ok(a.meta, CHECK_EDGE_PTR, e1, (long long)a.n_edges + 1, pos) ||
                        !dbg_ok(a.meta, CHECK_EDGE_PTR, e1 - e0, (long long)a.n_edges + 1, pos)))
            e0 = e1 = 0;
        // 1024 columns per pass: a lane holds four 16-byte pieces 256 columns apart
        for (int pb = 0; pb < pieces; pb += 128) {
            float acc[4][8];
#pragma unroll
            for (int m = 0; m < 4; ++m)
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[m][i] = 0.f;
            const uint4* src = reinterpret_cast<const uint4*>(a.hb + (size_t)e0 * a.Hp) + pb + lane;
            for (int e = e0; e < e1; ++e, src += pieces) {
                uint4 w[4];
#pragma unroll
                for (int m = 0; m < 4; ++m) w[m] = (pb + m * 32 + lane < pieces) ? __ldcg(src + m * 32) : make_uint4(0, 0, 0, 0);
#pragma unroll
                for (int m = 0; m < 4; ++m) {
                    const uint32_t u[4] = {w[m].x, w[m].y, w[m].z, w[m].w};
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        acc[m][2 * i] += __uint_as_float(u[i] << 16);
                        acc[m][2 * i + 1] += __uint_as_float(u[i] & 0xffff0000u);
                    }
                }
            }
#pragma unroll
            for (int m = 0; m < 4; ++m) {
                if (pb + m * 32 + lane >= pieces) continue;
                uint32_t o[4];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    __nv_bfloat162 p2 = __floats2bfloat162_rn(acc[m][2 * i], acc[m][2 * i + 1]);
                    o[i] = *reinterpret_cast<uint32_t*>(&p2);
                }
                reinterpret_cast<uint4*>(a.hs + r * a.Hp)[pb + m * 32 + lane] = make_uint4(o[0], o[1], o[2], o[3]);
            }
        }
    }
}

// ---- the child-ordered layout ----------------------------------------------------------------------------------
// Edge slots: the children of the internal node at position p (row r = p - n_leaves) own slots eoff[r] .. eoff[r+1]-1 in
// child-list order, eoff being the running sum of the child counts over the rows.  Three small kernels: counts and a
// scan inside blocks of 1024 rows, a scan of the block totals, and the fill of the per-slot tables.
constexpr int SCAN_TB = 1024;

__global__ void __launch_bounds__(SCAN_TB) edge_count_kernel(TcArgs a, int32_t* block_sum) {
    __shared__ int wsum[32];
    griddep_wait();
    griddep_launch();
    const int n_levels = a.meta[META_N_LEVELS];
    const int n_leaves = n_levels > 0 ? a.level_ptr[1] : 0;
    const int n_int = a.n_nodes - n_leaves;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    const int r = blockIdx.x * SCAN_TB + threadIdx.x;
    if (blockIdx.x * SCAN_TB > n_int) return;  // the block holds none of the rows 0 .. n_int
    int cnt = 0;
    if (r < n_int) {
        const int v = a.perm[n_leaves + r];
        if (!a.debug || dbg_ok(a.meta, CHECK_PERM, v, a.n_nodes, n_leaves + r)) cnt = a.child_ptr[v + 1] - a.child_ptr[v];
        if (a.debug && !dbg_ok(a.meta, CHECK_EDGE_PTR, cnt, (long long)a.n_edges + 1, n_leaves + r)) cnt = 0;
    }
    int incl = cnt;
#pragma unroll
    for (int o = 1; o < 32; o <<= 1) {
        const int y = __shfl_up_sync(0xffffffffu, incl, o);
        if (lane >= o) incl += y;
    }
    if (lane == 31) wsum[w] = incl;
    __syncthreads();
    if (w == 0) {
        int t = wsum[lane];
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, t, o);
            if (lane >= o) t += y;
        }
        wsum[lane] = t;
    }
    __syncthreads();
    if (w > 0) incl += wsum[w - 1];
    if (r <= n_int) a.eoff[r] = incl - cnt;  // exclusive, inside the block (row n_int: the block's running total so far)
    if (threadIdx.x == SCAN_TB - 1) block_sum[blockIdx.x] = incl;
}

__global__ void __launch_bounds__(SCAN_TB) edge_scan_kernel(TcArgs a, int32_t* block_sum, int n_blocks_bound) {
    __shared__ int wsum[32];
    __shared__ int carry_s;
    griddep_wait();
    griddep_launch();
    const int n_levels = a.meta[META_N_LEVELS];
    const int n_leaves = n_levels > 0 ? a.level_ptr[1] : 0;
    const int n_int = a.n_nodes - n_leaves;
    int n_blocks = n_int / SCAN_TB + 1;  // blocks that hold a row 0 .. n_int
    if (n_blocks > n_blocks_bound) n_blocks = n_blocks_bound;
    const int lane = threadIdx.x & 31, w = threadIdx.x >> 5;
    if (threadIdx.x == 0) carry_s = 0;
    __syncthreads();
    for (int base = 0; base < n_blocks; base += SCAN_TB) {
        const int i = base + threadIdx.x;
        const int x = i < n_blocks ? block_sum[i] : 0;
        int incl = x;
#pragma unroll
        for (int o = 1; o < 32; o <<= 1) {
            const int y = __shfl_up_sync(0xffffffffu, incl, o);
            if (lane >= o) incl += y;
        }
        if (lane == 31) wsum[w] = incl;
        __syncthreads();
        if (w == 0) {
            int t = wsum[lane];
#pragma unroll
            for (int o = 1; o < 32; o <<= 1) {
                const int y = __shfl_up_sync(0xffffffffu, t, o);
                if (lane >= o) t += y;
            }
            wsum[lane] = t;
        }
        __syncthreads();
        if (w > 0) incl += wsum[w - 1];
        const int carry = carry_s;
        if (i < n_blocks) block_sum[i] = incl - x + carry;  // exclusive over the blocks
        __syncthreads();
        if (threadIdx.x == SCAN_TB - 1) carry_s = carry + incl;
        __syncthreads();
    }
}

// One warp per internal node: finishes eoff and files every child under its slot.
__global__ void __launch_bounds__(256) edge_fill_kernel(TcArgs a, const int32_t* block_sum) {
    griddep_wait();
    griddep_launch();
    const int n_levels = a.meta[META_N_LEVELS];
    const int n_leaves = n_levels > 0 ? a.level_ptr[1] : 0;
    const int n_int = a.n_nodes - n_leaves;
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    for (int r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r <= n_int; r += warps) {
        const int e0 = a.eoff[r] + block_sum[r / SCAN_TB];
        __syncwarp();
        if (lane == 0) a.eoff[r] = e0;
        if (r == n_int) continue;
        const int v = a.perm[n_leaves + r];
        if (a.debug && !dbg_ok(a.meta, CHECK_PERM, v, a.n_nodes, n_leaves + r)) continue;
        const int c0 = a.child_ptr[v], cnt = a.child_ptr[v + 1] - c0;
        for (int i = lane; i < cnt; i += 32) {
            const int k = a.child_idx[c0 + i], sl = e0 + i;
            if (a.debug && (!dbg_ok(a.meta, CHECK_CHILD, k, a.n_nodes, v) || !dbg_ok(a.meta, CHECK_SLOT, sl, a.n_edges, v))) continue;
            const int kp = a.inv[k];
            if (a.debug && !dbg_ok(a.meta, CHECK_POSITION, kp, a.n_nodes, k)) continue;
            a.slot_par[sl] = r;
            a.slot_child[sl] = k;
            a.slot_of_pos[kp] = sl;
        }
    }
}

// x in any accepted form -> bf16 rows in LEVEL order (row i = node perm[i]), Dp elements each (Dp multiple of 8,
// zero padded).  One pass over x; after it the input projection reads plain TMA tiles, leaves and internal nodes
// sit in separate row ranges, and a tile is re-read from L2, not gathered, by each of its N tiles.
// One warp per row; 16-byte accesses when the source allows them.
__global__ void __launch_bounds__(256) level_order_x_kernel(const void* __restrict__ x, int is_bf16, int64_t ldx,
                                                            const int32_t* __restrict__ perm, int N, int D, int Dp,
                                                            int vec_ok, __nv_bfloat16* __restrict__ out,
                                                            int32_t* __restrict__ inv, int32_t* meta, int debug) {
    griddep_wait();
    griddep_launch();
    const int lane = threadIdx.x & 31;
    const int warps = (gridDim.x * blockDim.x) >> 5;
    for (int pos = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; pos < N; pos += warps) {
        const int64_t v = perm[pos];
        if (debug && !dbg_ok(meta, CHECK_PERM, v, N, pos)) continue;
        if (inv && lane == 0) inv[v] = pos;  // where the node sits in level order
        __nv_bfloat16* dst = out + (size_t)pos * Dp;
        if (vec_ok) {  // bf16 source, 16-byte aligned rows
            const uint4* src = reinterpret_cast<const uint4*>((const __nv_bfloat16*)x + v * ldx);
            for (int c = lane; c < Dp / 8; c += 32) {
                uint4 w = src[c];
                if (c * 8 + 8 > D) {  // zero the padding of the last chunk
                    __nv_bfloat16* e = reinterpret_cast<__nv_bfloat16*>(&w);
                    for (int i = 0; i < 8; ++i)
                        if (c * 8 + i >= D) e[i] = __float2bfloat16_rn(0.f);
                }
                reinterpret_cast<uint4*>(dst)[c] = w;
            }
        } else {
            for (int d = lane; d < Dp; d += 32) {
                float val = 0.f;
                if (d < D) val = is_bf16 ? __bfloat162float(((const __nv_bfloat16*)x)[v * ldx + d]) : ((const float*)x)[v * ldx + d];
                dst[d] = __float2bfloat16_rn(val);
            }
        }
    }
}

// Position of every node in level order (the inverse of perm), for forwards that do not copy x.
__global__ void __launch_bounds__(256) inverse_perm_kernel(const int32_t* __restrict__ perm, int N, int32_t* __restrict__ inv,
                                                           int32_t* meta, int debug) {
    griddep_wait();
    griddep_launch();
    for (int pos = blockIdx.x * blockDim.x + threadIdx.x; pos < N; pos += gridDim.x * blockDim.x) {
        const int v = perm[pos];
        if (debug && !dbg_ok(meta, CHECK_PERM, v, N, pos)) continue;
        inv[v] = pos;
    }
}

// ---- weight packing for the tensor-core path -----------------------------------------------------------
// Rows of B are output features; each 64-wide hidden slice keeps its gates next to each other so that one
// accumulator tile holds every gate of the same hidden indices: row n of a G-gate matrix maps to
// hidden index (n / (64 G)) * 64 + n % 64, gate (n % (64 G)) / 64.
__global__ void pack_tc_kernel(const float* __restrict__ src /*[4H, K]*/, int K, int H, int Hp, int Kp, int gates,
                               int gate_first, __nv_bfloat16* __restrict__ out /*[gates*Hp, Kp]*/) {
    const long long total = (long long)gates * Hp * Kp;
    for (long long idx = (long long)blockIdx.x * blockDim.x + threadIdx.x; idx < total;
         idx += (long long)gridDim.x * blockDim.x) {
        const int n = (int)(idx / Kp), k = (int)(idx - (long long)n * Kp);
        const int blk = n / (64 * gates), g = (n % (64 * gates)) / 64, j = blk * 64 + n % 64;
        float val = 0.f;
        if (j < H && k < K) val = src[((long long)(gate_first + g) * H + j) * K + k];
        out[idx] = __float2bfloat16_rn(val);
    }
}

__global__ void pack_bias_tc_kernel(const float* __restrict__ b, int H, int Hp, float* __restrict__ out) {
    int idx = blockIdx.x * blockDim.x + threadIdx.x;
    if (idx >= 4 * Hp) return;
    int j = idx >> 2, g = idx & 3;
    out[idx] = j < H ? b[g * H + j] : 0.f;
}

// ---- host side -------------------------------------------------------------------------------------------
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

EncodeTiledFn encode_fn() {
    static EncodeTiledFn fn = nullptr;
    if (!fn) {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess &&
            q == cudaDriverEntryPointSuccess)
            fn = (EncodeTiledFn)p;
    }
    return fn;
}

// bf16 row-major [rows, cols] with row stride ld (elements); box = 64 columns x box_rows, 128-byte swizzle
bool make_tmap(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint64_t ld, uint32_t box_rows) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 2};
    cuuint32_t box[2] = {64, box_rows};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// fp32 row-major [rows, cols] with row stride ld (elements); box = 32 columns x 32 rows, 128-byte swizzle (stores of P)
bool make_tmap_f32(CUtensorMap* m, const void* base, uint64_t rows, uint64_t cols, uint64_t ld) {
    EncodeTiledFn fn = encode_fn();
    if (!fn) return false;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {ld * 4};
    cuuint32_t box[2] = {32, 32};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(m, CU_TENSOR_MAP_DATA_TYPE_FLOAT32, 2, const_cast<void*>(base), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_NONE,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    return r == CUDA_SUCCESS;
}

// The switches of one forward call (jdb_opts.tuning, or the defaults with the environment's overrides, read at every
// call so that nothing depends on what an earlier call saw).
//   pair_mask  which GEMMs run as CTA pairs (cta_group::2) when they have enough 256-row tiles: 1 input projection,
//              2 level GEMM, 4 forget-gate GEMM.  Default 7 (the per-level GEMMs launch by launch, from 32 tiles per
//              pair on; the gate GEMM gains about 2 % on the wide forest): all gain from the pair reading half of B per SM, the
//              projection only together with eight epilogue warps (same-box runs on the wide forest: 10.9 ms as
//              pairs with eight warps, 11.7 as pairs with four, 11.4-11.6 as lone CTAs with four).
//   pdl        programmatic dependent launch of the forward kernels (each waits for its predecessor inside the
//              kernel, after its own set-up)
struct Tuning {
    int pair_mask, issuers;
    bool pdl, p_tma;
    bool issuers2_requested;   // two MMA issuers exist only in the kernels with four epilogue warps
    bool gather_x;             // read x in place through TMA row gathers instead of laying it out in level order first
    bool tree_groups;          // cooperative loop partitioned by tree (where possible)
};
Tuning resolve_tuning(int32_t t) {
    Tuning r;
    if (t & JDB_TUNE_SET) {
        r.pair_mask = ((t & JDB_TUNE_PAIR_XPROJ) ? 1 : 0) | ((t & JDB_TUNE_PAIR_LEVEL) ? 2 : 0) | ((t & JDB_TUNE_PAIR_FORGET) ? 4 : 0);
        r.issuers = (t & JDB_TUNE_TWO_ISSUERS) ? 2 : 1;
        r.pdl = !(t & JDB_TUNE_NO_PDL);
        r.p_tma = !(t & JDB_TUNE_PLAIN_STORES);
        r.issuers2_requested = r.issuers == 2;
        r.gather_x = (t & JDB_TUNE_GATHER_X) != 0;
        r.tree_groups = (t & JDB_TUNE_TREE_GROUPS) != 0;
        return r;
    }
    const char* e = getenv("JDB_GEMM_PAIR");
    r.pair_mask = e ? (atoi(e) & 7) : 7;
    e = getenv("JDB_GEMM_ISSUERS");
    r.issuers = (e && e[0] == '2') ? 2 : 1;
    e = getenv("JDB_PDL");
    r.pdl = !(e && e[0] == '0');
    e = getenv("JDB_P_TMA");
    r.p_tma = !(e && e[0] == '0');
    r.issuers2_requested = r.issuers == 2;
    e = getenv("JDB_GATHER_X");
    r.gather_x = e && e[0] == '1';
    e = getenv("JDB_TREE_GROUPS");
    r.tree_groups = e && e[0] == '1';
    return r;
}

template <class... KArgs, class... Args>
cudaError_t launch_behind(bool pdl, void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr[1];
    attr[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = attr;
    cfg.numAttrs = pdl ? 1 : 0;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

}  // namespace

TcPackLayout tc_pack_layout(int32_t D, int32_t H) {
    TcPackLayout L{};
    L.Hp = (H + 63) / 64 * 64;
    L.Kd = (D + 63) / 64 * 64;
    size_t off = 0;
    L.off_bias = off; off += align_up((size_t)L.Hp * 4 * sizeof(float), 256);
    L.off_W = off;    off += align_up((size_t)4 * L.Hp * L.Kd * 2, 256);
    L.off_Uiou = off; off += align_up((size_t)3 * L.Hp * L.Hp * 2, 256);
    L.off_Uf = off;   off += align_up((size_t)L.Hp * L.Hp * 2, 256);
    L.total = off;
    return L;
}

jdb_status tc_pack_weights_enqueue(const float* W, const float* U, const float* b, int32_t D, int32_t H, void* packed_tc,
                                   cudaStream_t st) {
    TcPackLayout L = tc_pack_layout(D, H);
    char* base = (char*)packed_tc;
    pack_bias_tc_kernel<<<ceil_div(4 * L.Hp, 256), 256, 0, st>>>(b, H, L.Hp, (float*)(base + L.off_bias));
    pack_tc_kernel<<<1024, 256, 0, st>>>(W, D, H, L.Hp, L.Kd, 4, 0, (__nv_bfloat16*)(base + L.off_W));
    pack_tc_kernel<<<1024, 256, 0, st>>>(U, H, H, L.Hp, L.Hp, 3, 0, (__nv_bfloat16*)(base + L.off_Uiou));
    pack_tc_kernel<<<1024, 256, 0, st>>>(U, H, H, L.Hp, L.Hp, 1, 3, (__nv_bfloat16*)(base + L.off_Uf));
    JDB_CUDA_TRY(cudaGetLastError());
    return JDB_OK;
}

namespace {
// carving of the forward workspace (the same walk sizes it and hands out the pieces)
struct TcWorkspace {
    float* P;
    __nv_bfloat16* hs;
    float* S;
    __nv_bfloat16* hb;
    __nv_bfloat16* xb;
    int32_t *inv, *eoff, *slot_of_pos, *slot_par, *slot_child, *block_sum;
    void* part_ws;   // tree partition of the cooperative loop (hidden sizes that kernel serves)
    size_t s_bytes, slot_of_pos_bytes, total;
    int n_scan_blocks;
};
TcWorkspace carve_tc_ws(void* ws, int32_t n_nodes, int32_t n_internal_bound, int32_t D, int32_t H, int Hp) {
    const size_t n = (size_t)(n_nodes > 0 ? n_nodes : 1), ni = (size_t)(n_internal_bound > 0 ? n_internal_bound : 1);
    char* p = (char*)ws;
    auto take = [&](size_t bytes) { char* q = p; p += align_up(bytes, 256); return q; };
    TcWorkspace w{};
    w.P = (float*)take(ni * Hp * 4 * sizeof(float));
    w.hs = (__nv_bfloat16*)take(ni * Hp * 2);
    w.s_bytes = ni * Hp * sizeof(float);
    w.S = (float*)take(w.s_bytes);
    w.hb = (__nv_bfloat16*)take(n * Hp * 2);
    w.xb = (__nv_bfloat16*)take(n * (size_t)((D + 7) / 8 * 8) * 2);
    w.inv = (int32_t*)take(n * sizeof(int32_t));
    w.eoff = (int32_t*)take((ni + 1 + SCAN_TB) * sizeof(int32_t));
    w.slot_of_pos_bytes = n * sizeof(int32_t);
    w.slot_of_pos = (int32_t*)take(w.slot_of_pos_bytes);
    w.slot_par = (int32_t*)take(n * sizeof(int32_t));
    w.slot_child = (int32_t*)take(n * sizeof(int32_t));
    w.n_scan_blocks = (int)(ni / SCAN_TB + 1);
    w.block_sum = (int32_t*)take((size_t)w.n_scan_blocks * sizeof(int32_t));
    w.part_ws = small_levels_supported(H) ? (void*)take(partition_ws_bytes(n_nodes)) : nullptr;
    w.total = (size_t)(p - (char*)ws);
    return w;
}
}  // namespace

size_t forward_tc_ws_bytes(int32_t n_nodes, int32_t n_internal_bound, int32_t D, int32_t H) {
    return carve_tc_ws(nullptr, n_nodes, n_internal_bound, D, H, tc_pack_layout(D, H).Hp).total;
}

jdb_status forward_tc_enqueue(const ForwardArgs& fa, const void* packed_tc, int n_levels, int n_internal_bound,
                              void* ws, bool use_small, uint64_t timeout_ns, cudaStream_t st) {
    const int N = fa.n_nodes, D = fa.D, H = fa.H;
    TcPackLayout L = tc_pack_layout(D, H);
    const int Hp = L.Hp;
    if (!encode_fn()) return JDB_ERR_UNSUPPORTED;
    DevInfo* di = dev_info();
    if (!di) return JDB_ERR_CUDA;
    const int n_sm = di->n_sm;

    const size_t n = (size_t)N, ni = (size_t)(n_internal_bound > 0 ? n_internal_bound : 1);
    const TcWorkspace w = carve_tc_ws(ws, N, n_internal_bound, D, H, Hp);
    const int Dp = (D + 7) / 8 * 8;

    const char* pk = (const char*)packed_tc;
    TcArgs a{};
    a.child_ptr = fa.child_ptr; a.child_idx = fa.child_idx; a.level_ptr = fa.level_ptr; a.perm = fa.perm;
    a.meta = fa.meta; a.n_nodes = N; a.n_edges = fa.n_edges; a.n_int_bound = (int32_t)ni; a.H = H; a.Hp = Hp;
    a.bias4 = (const float*)(pk + L.off_bias);
    a.P = w.P; a.S = w.S; a.hs = w.hs; a.hb = w.hb; a.inv = w.inv; a.h = fa.h; a.c = fa.c; a.ldh = fa.ldh;
    a.vec_ok = (fa.ldh % 4 == 0) && (((uintptr_t)fa.h & 15) == 0) && (((uintptr_t)fa.c & 15) == 0);
    a.child_order = use_small ? 0 : 1;
    a.eoff = w.eoff; a.slot_of_pos = w.slot_of_pos; a.slot_par = w.slot_par; a.slot_child = w.slot_child;
    a.debug = fa.debug;
    const Tuning tune = resolve_tuning(fa.tuning);
    a.issuers = tune.issuers;
    a.p_tma = tune.p_tma ? 1 : 0;

    // x goes into level order (and bf16) once, in a pass of its own; the copy reads 16-byte pieces when x is bf16 with
    // aligned rows.  Such an x can instead be read in place, its rows picked by perm through TMA row gathers
    // (JDB_TUNE_GATHER_X): correct, but every K block of every tile then costs 32 four-row gathers instead of one
    // box load, and the copy engine does not keep up (workload 5 projection 28.8 ms instead of 11.8, workload 3
    // 0.79 instead of 0.44), so it is off unless asked for.
    const int x_vec = fa.x_is_bf16 && (fa.ldx % 8 == 0) && (((uintptr_t)fa.x & 15) == 0);
    a.x_gather = (x_vec && tune.gather_x) ? 1 : 0;
    // CTA pairs pay off once there are enough 256-row tiles to keep every pair busy; below that the lone-CTA
    // kernel has the shorter tail.  In pair mode every CTA loads half of a B tile, so the B maps have half-height boxes.
    const bool big = !use_small && (long long)N >= 2LL * BM * n_sm;
    // the projection as pairs from about 128 tiles per pair on (1.57 M rows x 16 N tiles: 10.9 vs 11.5 ms; 143 k rows x 8:
    // 0.455 vs 0.444 ms, so that one stays with lone CTAs); an explicit tuning word decides by itself
    const long long x_tiles2 = ((long long)N + 2 * BM - 1) / (2 * BM) * (4LL * Hp / 256);
    const bool x_many = (fa.tuning & JDB_TUNE_SET) || x_tiles2 >= 128LL * (n_sm / 2);
    const bool pair_x = big && x_many && (tune.pair_mask & 1), pair_l = big && (tune.pair_mask & 2), pair_f = big && (tune.pair_mask & 4);
    const uint32_t bdiv = pair_x ? 2 : 1;
    CUtensorMap tmX, tmW, tmWl, tmHS, tmUiou, tmUiouh, tmHB, tmHBh, tmUf, tmP, tmHBs;
    // W is read through a full box and a leaf box (i, o, u blocks only)
    bool ok = (a.x_gather ? make_tmap(&tmX, fa.x, n, (uint64_t)D, (uint64_t)fa.ldx, 1)    // one-row boxes for the gathers
                          : make_tmap(&tmX, w.xb, n, (uint64_t)D, (uint64_t)Dp, BM)) &&
              make_tmap(&tmW, pk + L.off_W, (uint64_t)4 * Hp, (uint64_t)L.Kd, (uint64_t)L.Kd, 256 / bdiv) &&
              make_tmap(&tmWl, pk + L.off_W, (uint64_t)4 * Hp, (uint64_t)L.Kd, (uint64_t)L.Kd, 192 / bdiv);
    if (ok && !use_small)   // the per-level launches read their operands through six more maps
        ok = make_tmap(&tmHS, w.hs, ni, (uint64_t)Hp, (uint64_t)Hp, BM) &&
             make_tmap(&tmUiou, pk + L.off_Uiou, (uint64_t)3 * Hp, (uint64_t)Hp, (uint64_t)Hp, 192) &&
             make_tmap(&tmUiouh, pk + L.off_Uiou, (uint64_t)3 * Hp, (uint64_t)Hp, (uint64_t)Hp, 96) &&   // half per CTA of a pair
             make_tmap(&tmHB, w.hb, n, (uint64_t)Hp, (uint64_t)Hp, F_EDGES) &&        // forget-gate GEMM: B, a tile's 256 edge rows
             make_tmap(&tmHBh, w.hb, n, (uint64_t)Hp, (uint64_t)Hp, F_EDGES / 2) &&   // ... half of them per CTA of a pair
             make_tmap(&tmUf, pk + L.off_Uf, (uint64_t)Hp, (uint64_t)Hp, (uint64_t)Hp, BM);   // ... A, 128 hidden units
    ok = ok && make_tmap_f32(&tmP, w.P, ni, (uint64_t)4 * Hp, (uint64_t)4 * Hp) &&
         make_tmap(&tmHBs, w.hb, n, (uint64_t)Hp, (uint64_t)Hp, 32);  // store boxes: 64 columns x one warp's 32 rows
    if (!ok) return JDB_ERR_UNSUPPORTED;

    if (!(di->attr_mask & ATTR_GEMM_TC)) {
        JDB_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<EPI_XPROJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_STORE));
        JDB_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<EPI_LEVEL>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_LEVEL));
        JDB_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<EPI_F>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_F));
        JDB_CUDA_TRY(cudaFuncSetAttribute(gemm_tc_kernel<EPI_XPROJ8>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM_SMEM_X8));
        JDB_CUDA_TRY(cudaFuncSetAttribute(gemm_tc2_kernel<EPI_XPROJ8>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM2_SMEM_X8));
        JDB_CUDA_TRY(cudaFuncSetAttribute(gemm_tc2_kernel<EPI_XPROJ>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM2_SMEM));
        JDB_CUDA_TRY(cudaFuncSetAttribute(gemm_tc2_kernel<EPI_LEVEL>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM2_SMEM_LEVEL));
        JDB_CUDA_TRY(cudaFuncSetAttribute(gemm_tc2_kernel<EPI_F>, cudaFuncAttributeMaxDynamicSharedMemorySize, GEMM2_SMEM_F));
        di->attr_mask |= ATTR_GEMM_TC;
    }

    auto gemm_grid = [&](long long rows_bound, int n_tiles) {
        long long tiles = (rows_bound + BM - 1) / BM * n_tiles;
        return (int)(tiles < n_sm ? (tiles > 0 ? tiles : 1) : n_sm);
    };
    const int kd = L.Kd / BK, kh = Hp / BK;

    TcArgs af = a;   // the forget-gate GEMM always has one MMA issuer (its warps 2-9 are all epilogue warps)
    af.issuers = 1;
    // one GEMM launch: a lone-CTA grid, or a grid of CTA pairs (clusters of 2) for launches with many tiles
    auto launch = [&](int epi, const CUtensorMap& tA, const CUtensorMap& tB_full, const CUtensorMap& tBl, long long rows_bound,
                      int level, int bn, int n_total, int kblocks) -> jdb_status {
        // tiles along the second dimension: N tiles of the weights, or (forget-gate GEMM) tiles of hidden units
        const int n_tiles = epi == EPI_F ? (Hp + BM - 1) / BM : n_total / bn;
        const int n_tiles2 = epi == EPI_F ? (Hp + 2 * BM - 1) / (2 * BM) : n_tiles;
        // the forget-gate GEMM decides launch by launch: pairs pay off from about 32 tiles per pair on
        const long long tiles2 = (rows_bound + 2 * BM - 1) / (2 * BM) * n_tiles2;
        const bool pair = is_xproj(epi) ? pair_x : ((epi == EPI_LEVEL ? pair_l : pair_f) && tiles2 >= 32LL * (n_sm / 2));
        const CUtensorMap& tB = (epi == EPI_F && pair) ? tmHBh : (epi == EPI_LEVEL && pair) ? tmUiouh : tB_full;
        if (!pair) {
            const long long lone_tiles = epi == EPI_F ? (rows_bound + F_EDGES - 1) / F_EDGES * n_tiles : 0;
            const int grid = epi == EPI_F ? (int)(lone_tiles < n_sm ? (lone_tiles > 0 ? lone_tiles : 1) : n_sm) : gemm_grid(rows_bound, n_tiles);
            if (epi == EPI_XPROJ) JDB_CUDA_TRY(launch_behind(tune.pdl, gemm_tc_kernel<EPI_XPROJ>, dim3(grid), dim3(GEMM1_THREADS), GEMM_SMEM_STORE, st, tA, tB, tBl, tmP, tmHBs, a, level, bn, n_total, kblocks));
            else if (epi == EPI_XPROJ8) JDB_CUDA_TRY(launch_behind(tune.pdl, gemm_tc_kernel<EPI_XPROJ8>, dim3(grid), dim3(GEMMF_THREADS), GEMM_SMEM_X8, st, tA, tB, tBl, tmP, tmHBs, af, level, bn, n_total, kblocks));
            else if (epi == EPI_LEVEL) JDB_CUDA_TRY(launch_behind(tune.pdl, gemm_tc_kernel<EPI_LEVEL>, dim3(grid), dim3(GEMM1_THREADS), GEMM_SMEM_LEVEL, st, tA, tB, tBl, tmP, tmHBs, a, level, bn, n_total, kblocks));
            else JDB_CUDA_TRY(launch_behind(tune.pdl, gemm_tc_kernel<EPI_F>, dim3(grid), dim3(GEMMF_THREADS), GEMM_SMEM_F, st, tA, tB, tBl, tmP, tmHBs, af, level, bn, n_total, kblocks));
            return JDB_OK;
        }
        int pairs = (int)(tiles2 < n_sm / 2 ? (tiles2 > 0 ? tiles2 : 1) : n_sm / 2);
        cudaLaunchConfig_t cfg{};
        cfg.gridDim = dim3(2 * pairs);
        cfg.blockDim = dim3(gemm2_threads(epi));
        cfg.dynamicSmemBytes = epi == EPI_LEVEL ? GEMM2_SMEM_LEVEL : epi == EPI_F ? GEMM2_SMEM_F : epi == EPI_XPROJ8 ? GEMM2_SMEM_X8 : GEMM2_SMEM;
        cfg.stream = st;
        cudaLaunchAttribute attr[2];
        attr[0].id = cudaLaunchAttributeClusterDimension;
        attr[0].val.clusterDim.x = 2;
        attr[0].val.clusterDim.y = 1;
        attr[0].val.clusterDim.z = 1;
        attr[1].id = cudaLaunchAttributeProgrammaticStreamSerialization;
        attr[1].val.programmaticStreamSerializationAllowed = 1;
        cfg.attrs = attr;
        cfg.numAttrs = tune.pdl ? 2 : 1;
        if (epi == EPI_XPROJ) JDB_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<EPI_XPROJ>, tA, tB, tBl, tmP, tmHBs, a, level, bn, n_total, kblocks));
        else if (epi == EPI_XPROJ8) JDB_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<EPI_XPROJ8>, tA, tB, tBl, tmP, tmHBs, af, level, bn, n_total, kblocks));
        else if (epi == EPI_LEVEL) JDB_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<EPI_LEVEL>, tA, tB, tBl, tmP, tmHBs, a, level, bn, n_total, kblocks));
        else JDB_CUDA_TRY(cudaLaunchKernelEx(&cfg, gemm_tc2_kernel<EPI_F>, tA, tB, tBl, tmP, tmHBs, af, level, bn, n_total, kblocks));
        return JDB_OK;
    };

    jdb_status ls = JDB_OK;
    if (fa.ev_begin) JDB_CUDA_TRY(cudaEventRecord(fa.ev_begin, st));
    if (a.x_gather) {
        const long long want = ((long long)N + 255) / 256;
        const int blocks = (int)(want < (long long)n_sm * 8 ? want : (long long)n_sm * 8);
        JDB_CUDA_TRY(launch_behind(tune.pdl, inverse_perm_kernel, dim3(blocks), dim3(256), 0, st, fa.perm, N, w.inv, fa.meta, (int)fa.debug));
    } else {
        const long long want = ((long long)N + 7) / 8;
        const int blocks = (int)(want < (long long)n_sm * 16 ? want : (long long)n_sm * 16);
        JDB_CUDA_TRY(launch_behind(tune.pdl, level_order_x_kernel, dim3(blocks), dim3(256), 0, st, fa.x, (int)fa.x_is_bf16, fa.ldx, fa.perm, N, D, Dp,
                                   (int)x_vec, w.xb, w.inv, fa.meta, (int)fa.debug));
    }
    if (!use_small) {
        // child-ordered layout: slots of the edges, and which slot every node's bf16 row goes to; S starts at zero
        JDB_CUDA_TRY(cudaMemsetAsync(w.slot_of_pos, 0xFF, w.slot_of_pos_bytes, st));
        JDB_CUDA_TRY(cudaMemsetAsync(w.S, 0, w.s_bytes, st));
        edge_count_kernel<<<w.n_scan_blocks, SCAN_TB, 0, st>>>(a, w.block_sum);
        edge_scan_kernel<<<1, SCAN_TB, 0, st>>>(a, w.block_sum, w.n_scan_blocks);
        const long long want = ((long long)ni + 1 + 7) / 8;
        edge_fill_kernel<<<(int)(want < (long long)n_sm * 16 ? want : (long long)n_sm * 16), 256, 0, st>>>(a, w.block_sum);
        JDB_CUDA_TRY(cudaGetLastError());
    }
    // Eight epilogue warps where the bf16 copy of h goes out row by row anyway (child order) and either K is short or
    // the GEMM runs as CTA pairs: with at most eight K blocks per tile the epilogue weighs more than the pipeline stage
    // the eight step buffers cost a lone CTA (D = 512: 0.47 -> 0.44 ms on 143 k nodes), while at sixteen K blocks the
    // lone four-stage kernel is ahead of the lone three-stage one (D = 1024: 1.16 vs 1.22 ms on 195 k nodes); a CTA of a
    // pair keeps four stages either way.  The small forests of the cooperative loop keep the four-warp kernel, whose
    // leaf tiles leave as one TMA box per warp.
    const int xepi = (!use_small && !tune.issuers2_requested && (kd <= 8 || pair_x)) ? EPI_XPROJ8 : EPI_XPROJ;
    if ((ls = launch(xepi, tmX, tmW, tmWl, (long long)N + 2 * BM, 0, 256, 4 * Hp, kd)) != JDB_OK) return ls;
    if (fa.ev_xproj_done) JDB_CUDA_TRY(cudaEventRecord(fa.ev_xproj_done, st));
    if (!use_small) {
        const int cs_blocks = (int)((ni + 7) / 8 < (size_t)n_sm * 8 ? (ni + 7) / 8 : (size_t)n_sm * 8);
        for (int level = 1; level < n_levels; ++level) {
            JDB_CUDA_TRY(launch_behind(tune.pdl, childsum_kernel, dim3(cs_blocks), dim3(256), 0, st, a, level));
            if ((ls = launch(EPI_F, tmUf, tmHB, tmHB, (long long)fa.n_edges, level, F_EDGES, F_EDGES, kh)) != JDB_OK) return ls;
            if ((ls = launch(EPI_LEVEL, tmHS, tmUiou, tmUiou, (long long)ni, level, 192, 3 * Hp, kh)) != JDB_OK) return ls;
        }
        JDB_CUDA_TRY(cudaGetLastError());
    } else {
        // On request (JDB_TUNE_TREE_GROUPS) the forest is partitioned by tree: every group of CTAs then walks its own
        // trees and never waits for the rest of the grid.  The partition costs seven small launches and needs the level
        // count on the host (to size its table) and the depths.  Measured on the deep forest (230 k nodes, 87 levels):
        // level loop 1.17 ms against 1.12 ms with grid-wide barriers, the same bits: what bounds that loop is the chain
        // of dependent steps inside a pass (gather, product, read-out, stores) times the passes a group has to walk,
        // not the barrier between levels, so it stays off by default.
        Partition part{nullptr, nullptr, nullptr, 0};
        const int groups = small_levels_groups(H, n_internal_bound);
        const bool want = tune.tree_groups;
        if (want && fa.depth && n_levels > 2 && groups > 1 && N <= (1 << 21) && (long long)n_levels * groups <= PARTITION_TABLE_MAX &&
            groups <= PARTITION_MAX_GROUPS) {
            jdb_status s = partition_enqueue(fa, fa.depth, n_levels, groups, w.part_ws, &part, st);
            if (s != JDB_OK) return s;
        }
        jdb_status s = small_levels_enqueue(fa, packed_tc, w.P, w.hb, w.inv, n_internal_bound, 1, timeout_ns, part, st);
        if (s != JDB_OK) return s;
    }
    if (fa.ev_levels_done) JDB_CUDA_TRY(cudaEventRecord(fa.ev_levels_done, st));
    return JDB_OK;
}

}  // namespace jdb
