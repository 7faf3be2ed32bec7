// Level loop for small hidden sizes (H <= 192) in ONE cooperative launch: the persistent-kernel mode for
// forests whose levels are too small to amortise launches (deep, skewed trees; a batch of 256 short sentences).
//
// Every CTA owns a slice of 32 hidden units for the whole call and keeps that slice of U (96 rows of the i, o, u
// blocks and 32 forget rows, bf16) resident in shared memory as ONE tensor-core operand of 128 rows.  The unit of
// work is a pass: up to 128 child edges of a tile of NT nodes of one level.  Per pass the CTA
//   1. gathers the bf16 rows h_k of the pass's children straight into the other tensor-core operand (16-byte
//      asynchronous copies into the swizzled layout: no staging, no conversion) and this CTA's slice of every c_k;
//   2. issues tcgen05.mma once: [edges x 128] = h_k [U_iou ; U_f]^T for its 32 hidden units.  The i, o, u
//      columns of an edge row are that child's share of U_iou h~ (h~ = sum_k h_k is never formed: the sum moves
//      behind the product and is taken in fp32), the forget columns are U_f h_k;
//   3. reads TMEM back with all sixteen warps (lane quarter = warp % 4, gate block = warp / 4), turns the forget
//      columns into f_jk c_k = sig(P_f[j] + .) c_k, and passes everything through shared memory to
//   4. one thread per (node, hidden unit), which adds up the node's edge rows, adds the input projection,
//      finishes c_j = i u + sum_k f_jk c_k, h_j = o tanh(c_j) and stores c, h (fp32, node order) and the bf16
//      copy of h (level order) that the next level gathers.
// Nothing in a pass's description (node ids, child ids and positions, parent row of every edge, forget slices
// of the input projection) depends on h or c, so four extra warps prepare the descriptions ahead of the
// arithmetic, through a two-slot ring guarded by mbarriers; the chain of dependent index loads never sits
// between two tensor-core passes.  Levels are separated by a bounded grid barrier among the CTAs that have work.
#include "small_common.cuh"

namespace jdb {

namespace {

using namespace ptx;
using namespace small;

constexpr int SBJ = 32;            // hidden units per CTA
constexpr int SMAX_KB = 3;         // K blocks of 64 -> H <= 192
constexpr int ET = 128;            // edges per pass (the MMA's M)
constexpr int RPT = NT_MAX / MAIN_WARPS;  // tile rows per arithmetic thread in the cell arithmetic, at most
constexpr int KB_BYTES = 128 * 128;  // one K block of an operand: 128 rows of 128 bytes
constexpr int XLD = 132;           // floats per row of the exchange buffer (conflict-free 16-byte row writes)
constexpr int CS_LD = SBJ + 4;     // floats per staged c_k slice
constexpr int PF_LD = SBJ + 4;     // floats per staged forget slice of the input projection
constexpr int OFF_B = 0;                                  // [KB][128 rows][128 B]: rows 0-95 i,o,u; 96-127 forget
constexpr int OFF_A = OFF_B + SMAX_KB * KB_BYTES;         // [KB][128 edges][128 B]
constexpr int OFF_X = OFF_A + SMAX_KB * KB_BYTES;         // fp32 [128 edges][XLD]
constexpr int OFF_CS = OFF_X + ET * XLD * 4;              // fp32 [128 edges][CS_LD]
constexpr int OFF_PF = OFF_CS + ET * CS_LD * 4;           // fp32 [2][NT_MAX][PF_LD]
constexpr int SMALL_SMEM = OFF_PF + 2 * NT_MAX * PF_LD * 4 + 1024;
constexpr int S_TMEM_COLS = 128;   // columns 0-95: i, o, u shares of the edge rows; 96-127: their forget products
static_assert(SMALL_SMEM <= 220 * 1024, "shared memory budget");
static_assert(ET <= ET_MAX, "pass size");

struct SmallArgs {
    const int32_t* child_ptr;
    const int32_t* child_idx;
    const int32_t* level_ptr;
    const int32_t* perm;
    const int32_t* inv;         // position of every node in level order
    int32_t* meta;
    int32_t H, Hp, n_slices;
    const __nv_bfloat16* Uiou;  // [3 Hp][Hp], gates interleaved per 64-wide hidden block
    const __nv_bfloat16* Uf;    // [Hp][Hp]
    const float* P;             // [n_internal][4][Hp], planes i, o, u, f, rows in level order
    __nv_bfloat16* hb;          // [n_nodes][Hp] bf16 copy of h, rows in level order
    float* h;
    float* c;
    int64_t ldh;
    int32_t vec_ok;
    unsigned long long timeout_ns;
    int32_t first_level;  // levels below it were evaluated by launches of their own
    int32_t n_nodes, n_edges;
    int32_t debug;        // check every index against its array before following it
    // tree partition (G > 0: the launch has exactly G groups; each walks its own trees and synchronises inside the group)
    const int32_t* gperm;
    const int32_t* goff;
    int32_t* gbar;
    int32_t G;
    unsigned long long* trace;
    long long trace_cap;
};

__global__ void __launch_bounds__(STHREADS, 1) small_levels_kernel(SmallArgs a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ uint64_t bar_mma;
    __shared__ uint32_t s_tmem_base;
    __shared__ int s_abort, s_max_tiles;
    __shared__ Ring ring;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* sm = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const uint32_t sm_addr = smem_u32(sm);
    const int H = a.H, Hp = a.Hp, KB = Hp >> 6;
    const int slice = blockIdx.x % a.n_slices, grp = blockIdx.x / a.n_slices, n_grp = gridDim.x / a.n_slices;
    const int j0 = slice * SBJ;
    const int gather_chunks = a.n_slices * (SBJ / 8);  // 16-byte pieces of a bf16 row that carry hidden units
    float* xch = reinterpret_cast<float*>(sm + OFF_X);
    float* cs = reinterpret_cast<float*>(sm + OFF_CS);
    float* pfs = reinterpret_cast<float*>(sm + OFF_PF);

    if (tid == 0) {
        s_abort = 0;
        s_max_tiles = 1;
        mbar_init(smem_u32(&bar_mma), 1);
        ring_init(ring);
        fence_barrier_init();
    }
    if (warp == 0) tmem_alloc(smem_u32(&s_tmem_base), S_TMEM_COLS);
    for (int i = tid; i < (int)(2 * sizeof(PassSlot) / 4); i += STHREADS) reinterpret_cast<int*>(ring.slot)[i] = 0;
    // the edge operand starts as zeros: its columns past the last hidden slice are never written again
    for (int i = tid; i < SMAX_KB * KB_BYTES / 16; i += STHREADS) reinterpret_cast<uint4*>(sm + OFF_A)[i] = make_uint4(0, 0, 0, 0);

    // resident weight slice: operand row n = gate n / 32 (i, o, u, f), hidden unit j0 + n % 32
    for (int idx = tid; idx < KB * 4 * SBJ * 8; idx += STHREADS) {
        const int chunk = idx & 7, n = (idx >> 3) % (4 * SBJ), kb = idx / (8 * 4 * SBJ);
        const int g = n / SBJ, j = j0 + n % SBJ;
        const __nv_bfloat16* src = g < 3 ? a.Uiou + (size_t)((j >> 6) * 192 + g * 64 + (j & 63)) * Hp : a.Uf + (size_t)j * Hp;
        cp_async16(sm_addr + OFF_B + kb * KB_BYTES + n * 128 + ((chunk ^ (n & 7)) << 4), src + kb * 64 + chunk * 8);
    }
    cp_async_wait_all();
    fence_proxy_async();
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem_base = s_tmem_base;
    volatile int* abort = &s_abort;

    const int n_levels = a.meta[META_N_LEVELS];
    const bool bad_forest = a.meta[META_ERROR] != 0 || a.meta[META_UNFINISHED] != 0;
    const int n_leaves = n_levels > 0 ? a.level_ptr[1] : 0;
    bool alive = !bad_forest;
    // Tiles of 64 nodes halve the passes of a level with many tiles when most nodes have a single child (a pass
    // holds 128 edges); with more children per node a 64-node tile would need a second pass, so those forests keep
    // 32-node tiles everywhere.
    const int nt_max = (double)a.n_edges <= 1.35 * (double)(a.n_nodes - n_leaves) ? 64 : 32;

    // Only as many tile groups as the largest level has tiles take part; the others leave before the first
    // barrier, which therefore counts the participating CTAs only.
    {
        int mt = 1;
        for (int l = a.first_level + tid; l < n_levels; l += STHREADS) {
            int llo, lhi;
            checked_level(a.level_ptr, l, a.n_nodes, a.meta, a.debug, llo, lhi);
            const int ln = lhi - llo, nt = tile_nodes(ln, nt_max, n_grp);
            mt = max(mt, (ln + nt - 1) / nt);
        }
        if (mt > 1) atomicMax(&s_max_tiles, mt);
    }
    __syncthreads();
    const bool grouped = a.G > 0;   // every group takes part: it owns trees of its own
    const int active_grp = grouped ? n_grp : min(n_grp, s_max_tiles);
    const unsigned active_ctas = (unsigned)(active_grp * a.n_slices);
    if (grp >= active_grp) alive = false;

    if (warp >= MAIN_WARPS) {
        // ================= description warps: run ahead of the arithmetic by up to two passes =================
        if (alive) {
            DescribeArgs d{a.child_ptr, a.child_idx, a.level_ptr, a.perm, a.inv, a.first_level, n_levels, grp, n_grp, active_grp, nt_max,
                           a.meta, a.n_nodes, a.n_edges, a.debug, a.gperm, a.goff, a.G, n_leaves};
            describe_passes(d, ring, ET, abort, tid - MAIN_THREADS, [&](const PassSlot& S, int m, int tcount, int tm) {
                // forget slices of the tile's input projection, for this CTA's hidden units (parity selects the buffer)
                float* dst = pfs + (tcount & 1) * (NT_MAX * PF_LD);
                for (int task = tm; task < m * (SBJ / 4); task += META_THREADS) {
                    const int r = task >> 3, q = task & 7;
                    cp_async16(smem_u32(dst + r * PF_LD + 4 * q), a.P + ((size_t)S.prow[r] * 4 + 3) * Hp + j0 + 4 * q);
                }
            });
        }
    } else {
        // ================= arithmetic warps =================
        // level trace: thread 0 of CTA 0 stamps its first pass of each level
        auto stamp = [&](int level, int s, bool first) {
            if (a.trace && first && blockIdx.x == 0 && tid == 0 && (long long)level * 8 + s < a.trace_cap)
                a.trace[level * 8 + s] = global_ns();
        };
        const int quarter = warp & 3, gate = warp >> 2;  // TMEM lane quarter and gate block this warp reads out
        const int erow = quarter * 32 + lane;           // its edge row
        const uint32_t taddr = tmem_base + ((uint32_t)(quarter * 32) << 16) + (uint32_t)(gate * SBJ);
        uint32_t mma_phase = 0;
        int k = 0, tcount = 0;
        const DescribeArgs dm{a.child_ptr, a.child_idx, a.level_ptr, a.perm, a.inv, a.first_level, n_levels, grp, n_grp, active_grp, nt_max,
                              a.meta, a.n_nodes, a.n_edges, a.debug, a.gperm, a.goff, a.G, n_leaves};
        for (int level = a.first_level; level < n_levels && alive; ++level) {
            int lo, hi;
            group_level(dm, level, lo, hi);   // the same ranges and tiles as the description warps walk
            const int nt = tile_nodes(hi - lo, nt_max, grouped ? 1 : n_grp);
            const int tiles = (hi - lo + nt - 1) / nt;
            stamp(level, 0, true);
            const int tile0 = grouped ? 0 : grp, tile_step = grouped ? 1 : active_grp;
            for (int tile = tile0; tile < tiles && alive; tile += tile_step, ++tcount) {
                const bool first = tile == tile0;
                float zi[RPT], zo[RPT], zu[RPT], sfc[RPT];  // running sums of this thread's (row, hidden unit) pairs
#pragma unroll
                for (int i = 0; i < RPT; ++i) zi[i] = zo[i] = zu[i] = sfc[i] = 0.f;
                bool last = false;
                while (!last) {
                    const int s = k & 1;
                    const bool good = mbar_wait_warp(smem_u32(&ring.bar_full[s]), (uint32_t)((k >> 1) & 1), abort);
                    if (!good) *abort = 1;
                    const PassSlot& S = ring.slot[s];
                    const int m = S.m, ne = S.ne, et0 = S.et0;
                    const int nc = good ? min(ET, ne - et0) : 0;
                    last = !good || et0 + ET >= ne;
                    stamp(level, 1, first && et0 == 0);
                    // ---- gather: bf16 child rows into the operand, c slices beside it ----
                    for (int e = warp; e < nc; e += MAIN_WARPS) {
                        if (lane < gather_chunks)
                            cp_async16(sm_addr + OFF_A + (lane >> 3) * KB_BYTES + e * 128 + (((lane & 7) ^ (e & 7)) << 4),
                                       a.hb + (size_t)S.ek_pos[e] * Hp + lane * 8);
                    }
                    for (int task = tid; task < nc * (SBJ / 4); task += MAIN_THREADS) {
                        const int e = task >> 3, q = task & 7;
                        const float* crow = a.c + (int64_t)S.ek_id[e] * a.ldh;
                        if (a.vec_ok && j0 + 4 * q + 4 <= H) cp_async16(smem_u32(cs + e * CS_LD + 4 * q), crow + j0 + 4 * q);
                        else *reinterpret_cast<float4*>(cs + e * CS_LD + 4 * q) = load_row4(crow, j0 + 4 * q, H, a.vec_ok);
                    }
                    cp_async_wait_all();
                    fence_proxy_async();
                    if (named_bar_any(BAR_MAIN, MAIN_THREADS, !good || s_abort != 0)) { alive = false; break; }  // one verdict for all warps
                    stamp(level, 2, first && et0 == 0);
                    // ---- tensor cores: one product for all four gate blocks ----
                    if (tid == 0) {
                        tc_fence_after();
                        const uint32_t idesc = idesc_bf16(128, 4 * SBJ);
                        const int ksteps = a.n_slices * (SBJ / 16);  // K steps of 16 that carry hidden units
                        for (int ks = 0; ks < ksteps; ++ks) {
                            const int kb = ks >> 2, kk = ks & 3;
                            const uint64_t ad = smem_desc_sw128(sm_addr + OFF_A + kb * KB_BYTES);
                            const uint64_t bd = smem_desc_sw128(sm_addr + OFF_B + kb * KB_BYTES);
                            mma_bf16(tmem_base, ad + 2 * kk, bd + 2 * kk, idesc, ks != 0);
                        }
                        mma_commit(smem_u32(&bar_mma));
                    }
                    // input projection of this thread's pairs, on its way while the tensor cores run
                    float pi[RPT], po[RPT], pu[RPT];
#pragma unroll
                    for (int i = 0; i < RPT; ++i) {
                        const int r = warp + MAIN_WARPS * i;
                        pi[i] = po[i] = pu[i] = 0.f;
                        if (last && r < m) {
                            const float* prow = a.P + (size_t)S.prow[r] * 4 * Hp + j0 + lane;
                            pi[i] = __ldg(prow);
                            po[i] = __ldg(prow + Hp);
                            pu[i] = __ldg(prow + 2 * Hp);
                        }
                    }
                    const bool mma_done = mbar_wait_warp(smem_u32(&bar_mma), mma_phase, abort);
                    if (!mma_done) *abort = 1;
                    mma_phase ^= 1u;
                    tc_fence_after();
                    stamp(level, 4, first && et0 == 0);
                    // ---- accumulator read-out: 32 columns of one gate block for one edge row per thread ----
                    {
                        float v0[16], v1[16];
                        tmem_ld16(taddr, v0);
                        tmem_ld16(taddr + 16, v1);
                        tmem_ld_wait();
                        if (erow < nc) {
                            float* dst = xch + erow * XLD + gate * SBJ;
                            if (gate < 3) {
#pragma unroll
                                for (int q = 0; q < 4; ++q) {
                                    *reinterpret_cast<float4*>(dst + 4 * q) = make_float4(v0[4 * q], v0[4 * q + 1], v0[4 * q + 2], v0[4 * q + 3]);
                                    *reinterpret_cast<float4*>(dst + 16 + 4 * q) = make_float4(v1[4 * q], v1[4 * q + 1], v1[4 * q + 2], v1[4 * q + 3]);
                                }
                            } else {
                                const float4* pfrow = reinterpret_cast<const float4*>(pfs + (tcount & 1) * (NT_MAX * PF_LD) + S.ep[erow] * PF_LD);
                                const float4* ckrow = reinterpret_cast<const float4*>(cs + erow * CS_LD);
#pragma unroll
                                for (int q = 0; q < 8; ++q) {
                                    const float4 pf = pfrow[q], ck = ckrow[q];
                                    const float* f = q < 4 ? &v0[4 * q] : &v1[4 * (q - 4)];
                                    *reinterpret_cast<float4*>(dst + 4 * q) =
                                        make_float4(sigmoid_fast(pf.x + f[0]) * ck.x, sigmoid_fast(pf.y + f[1]) * ck.y,
                                                    sigmoid_fast(pf.z + f[2]) * ck.z, sigmoid_fast(pf.w + f[3]) * ck.w);
                                }
                            }
                        }
                    }
                    tc_fence_before();
                    if (named_bar_any(BAR_MAIN, MAIN_THREADS, !mma_done || s_abort != 0)) { alive = false; break; }
                    stamp(level, 5, first && et0 == 0);
                    // ---- cell arithmetic: one thread per (row, hidden unit) ----
#pragma unroll
                    for (int i = 0; i < RPT; ++i) {
                        const int r = warp + MAIN_WARPS * i;
                        if (r >= m) continue;
                        const int ea = max(S.eoff[r], et0), eb = min(S.eoff[r + 1], et0 + ET);
                        for (int e = ea; e < eb; ++e) {  // CSR order
                            const float* src = xch + (e - et0) * XLD + lane;
                            zi[i] += src[0];
                            zo[i] += src[SBJ];
                            zu[i] += src[2 * SBJ];
                            sfc[i] += src[3 * SBJ];
                        }
                        if (last) {
                            const float cc = fmaf(sigmoid_fast(zi[i] + pi[i]), tanh_fast(zu[i] + pu[i]), sfc[i]);
                            const float hh = sigmoid_fast(zo[i] + po[i]) * tanh_fast(cc);
                            const int vnode = S.nodes[r];
                            if (vnode < 0) continue;  // a row whose node id failed the debug checks
                            if (j0 + lane < H) {
                                a.c[(int64_t)vnode * a.ldh + j0 + lane] = cc;
                                a.h[(int64_t)vnode * a.ldh + j0 + lane] = hh;
                            }
                            // bf16 copy in level order: two hidden units per 4-byte store (padding columns hold exact zeros)
                            const __nv_bfloat16 hb16 = __float2bfloat16_rn(hh);
                            const unsigned mine = (unsigned)__bfloat16_as_ushort(hb16);
                            const unsigned next = __shfl_down_sync(0xffffffffu, mine, 1);
                            if ((lane & 1) == 0)
                                *reinterpret_cast<uint32_t*>(a.hb + (size_t)(S.prow[r] + n_leaves) * Hp + j0 + lane) = mine | (next << 16);
                        }
                    }
                    named_bar(BAR_MAIN, MAIN_THREADS);  // exchange buffer, operand and slot are free again
                    if (tid == 0) mbar_arrive(smem_u32(&ring.bar_empty[s]));
                    stamp(level, 6, first && last);
                    ++k;
                }
            }
            if (!alive) break;
            if (level + 1 < n_levels) {
                // all participating CTAs meet, or (tree partition) the CTAs of this group only
                int32_t* counter = grouped ? &a.gbar[grp] : &a.meta[META_BARRIER];
                const unsigned per_level = grouped ? (unsigned)a.n_slices : active_ctas;
                if (!main_grid_barrier(a.meta, counter, (unsigned)(level - a.first_level + 1) * per_level, a.timeout_ns, abort, tid)) alive = false;
            }
            stamp(level, 7, true);
        }
    }

    __syncthreads();
    if (s_abort && tid == 0) atomicExch(&a.meta[META_TIMEOUT], 1);
    tc_fence_after();
    if (warp == 0) tmem_dealloc(tmem_base, S_TMEM_COLS);
}

}  // namespace

bool small_levels_supported(int32_t H) { return H <= SMAX_KB * 64; }

int small_levels_groups(int32_t H, int n_internal_bound) {
    if (!small_levels_supported(H)) return 0;
    DevInfo* di = dev_info();
    if (!di) return 0;
    const int n_slices = (H + SBJ - 1) / SBJ;
    int groups = di->n_sm / n_slices;  // one CTA per SM: the kernel uses most of an SM's shared memory
    const int max_tiles = ceil_div(n_internal_bound > 0 ? n_internal_bound : 1, 32);
    if (groups > max_tiles) groups = max_tiles;
    return groups;
}

jdb_status small_levels_enqueue(const ForwardArgs& fa, const void* packed_tc, const float* P, void* hb, const int32_t* inv,
                                int n_internal_bound, int first_level, uint64_t timeout_ns, const Partition& part, cudaStream_t st) {
    const int H = fa.H;
    TcPackLayout L = tc_pack_layout(fa.D, H);
    if (!small_levels_supported(H)) return JDB_ERR_UNSUPPORTED;
    DevInfo* di = dev_info();
    if (!di) return JDB_ERR_CUDA;
    if (!(di->attr_mask & ATTR_SMALL_LEVELS)) {
        JDB_CUDA_TRY(cudaFuncSetAttribute(small_levels_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, SMALL_SMEM));
        di->attr_mask |= ATTR_SMALL_LEVELS;
    }
    if (di->small_per_sm == 0) {
        int per_sm = 0;
        JDB_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, small_levels_kernel, STHREADS, SMALL_SMEM));
        di->small_per_sm = per_sm > 0 ? 1 : -1;
    }
    if (di->small_per_sm < 1) return JDB_ERR_UNSUPPORTED;

    const char* pk = (const char*)packed_tc;
    SmallArgs a{};
    a.child_ptr = fa.child_ptr; a.child_idx = fa.child_idx; a.level_ptr = fa.level_ptr; a.perm = fa.perm;
    a.inv = inv;
    a.meta = fa.meta; a.H = H; a.Hp = L.Hp;
    a.n_slices = (H + SBJ - 1) / SBJ;
    a.Uiou = (const __nv_bfloat16*)(pk + L.off_Uiou);
    a.Uf = (const __nv_bfloat16*)(pk + L.off_Uf);
    a.P = P; a.hb = (__nv_bfloat16*)hb; a.h = fa.h; a.c = fa.c; a.ldh = fa.ldh;
    a.vec_ok = (fa.ldh % 4 == 0) && (((uintptr_t)fa.h & 15) == 0) && (((uintptr_t)fa.c & 15) == 0);
    a.timeout_ns = timeout_ns;
    a.first_level = first_level;
    a.trace = fa.trace;
    a.trace_cap = fa.trace_cap;

    a.n_nodes = fa.n_nodes; a.n_edges = fa.n_edges;
    a.debug = fa.debug;
    const int groups = small_levels_groups(H, n_internal_bound);
    if (groups < 1) return JDB_ERR_UNSUPPORTED;
    if (part.G > 0 && part.G != groups) return JDB_ERR_INVALID_ARG;   // the partition was made for another launch shape
    a.gperm = part.gperm; a.goff = part.goff; a.gbar = part.gbar; a.G = part.G;
    void* params[] = {&a};
    JDB_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)small_levels_kernel, dim3(groups * a.n_slices), dim3(STHREADS), params,
                                             SMALL_SMEM, st));
    return JDB_OK;
}

}  // namespace jdb
