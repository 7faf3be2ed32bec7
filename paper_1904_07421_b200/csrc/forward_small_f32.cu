// Level loop of the fp32 path (JDB_FP32, H <= 192) in ONE cooperative launch, on the plain FFMA units: the 1e-4
// bound of that path rules the tensor cores out.  Same organisation as the tensor-core loop of forward_small.cu:
// every CTA owns 32 hidden units for the whole call and keeps its slice of U (128 rows: i, o, u and forget rows
// of those units, fp32) resident in shared memory; the unit of work is a pass of up to 32 child edges of a tile of
// 4 to 32 nodes of one level (small levels are cut into small tiles so that every SM takes part); four extra warps
// describe the passes ahead of the arithmetic.  Per pass the CTA
//   1. gathers the fp32 rows h_k of the pass's children and this CTA's slice of every c_k (asynchronous copies);
//   2. computes [edges x 128] = h_k [U_iou ; U_f]^T with register tiles of 2 edges x 4 outputs per thread, reading
//      both operands from shared memory as 16-byte pieces along K (rows are an odd number of pieces apart, so the
//      eight rows a quarter-warp reads fall into different banks);
//   3. turns the forget columns into f_jk c_k = sig(P_f[j] + .) c_k and passes all four blocks through shared
//      memory to
//   4. one thread per (node, hidden unit): child sums in CSR order, c_j = i u + sum_k f_jk c_k, h_j = o tanh(c_j),
//      rows stored in node order.
// The K loop of every output runs in ascending k in one thread, so results do not depend on the launch shape.
#include "small_common.cuh"

namespace jdb {

namespace {

using namespace ptx;
using namespace small;

constexpr int SBJ = 32;       // hidden units per CTA
constexpr int FET = 32;       // edges per pass
constexpr int FNT = 32;       // nodes per tile, at most
constexpr int FNT_RULE = 0;   // tile_nodes() rule: 4 to 32 nodes, a level spread over all tile groups
constexpr int FMAX_H = 192;
constexpr int LDK = 49;       // 16-byte pieces per operand row (odd; 48 carry data for H = 192)
constexpr int LDF = 4 * LDK;  // floats per operand row
constexpr int XLD = 132;      // floats per row of the exchange buffer
constexpr int CS_LD = SBJ + 4;
constexpr int OFF_U = 0;                              // fp32 [128][LDF]: row n = gate n / 32, hidden unit j0 + n % 32
constexpr int OFF_HK = OFF_U + 128 * LDF * 4;         // fp32 [FET][LDF] child rows
constexpr int OFF_X = OFF_HK + FET * LDF * 4;         // fp32 [FET][XLD]
constexpr int OFF_CS = OFF_X + FET * XLD * 4;         // fp32 [FET][CS_LD]
constexpr int OFF_P = OFF_CS + FET * CS_LD * 4;       // float4 [2][FNT][SBJ]: input projection (i, o, u, f) of the tile
constexpr int F32_SMEM = OFF_P + 2 * FNT * SBJ * 16 + 1024;
static_assert(F32_SMEM <= 220 * 1024, "shared memory budget");

__device__ __forceinline__ float sigmoid_acc(float t) { return 1.0f / (1.0f + expf(-t)); }

struct F32Args {
    const int32_t* child_ptr;
    const int32_t* child_idx;
    const int32_t* level_ptr;
    const int32_t* perm;
    int32_t* meta;
    int32_t H, n_slices;
    int32_t n_nodes, n_edges;
    int32_t debug;       // check every index against its array before following it
    const float4* Ut4;   // [H][H]: Ut4[k * H + j] = (U_i, U_o, U_u, U_f)[j][k]
    const float4* P4;    // [n_internal][H]: biased input projection (i, o, u, f), rows in level order
    float* h;
    float* c;
    int64_t ldh;
    int32_t vec_ok;
    unsigned long long timeout_ns;
    unsigned long long* trace;
    long long trace_cap;
};

__global__ void __launch_bounds__(STHREADS, 1) small_levels_f32_kernel(F32Args a) {
    extern __shared__ uint8_t smem_raw[];
    __shared__ int s_abort, s_max_tiles;
    __shared__ Ring ring;

    const int tid = threadIdx.x, warp = tid >> 5, lane = tid & 31;
    uint8_t* sm = smem_raw + ((1024u - (smem_u32(smem_raw) & 1023u)) & 1023u);
    const int H = a.H, kq = (H + 3) >> 2;
    const int slice = blockIdx.x % a.n_slices, grp = blockIdx.x / a.n_slices, n_grp = gridDim.x / a.n_slices;
    const int j0 = slice * SBJ;
    float* us = reinterpret_cast<float*>(sm + OFF_U);
    float* hk = reinterpret_cast<float*>(sm + OFF_HK);
    float* xch = reinterpret_cast<float*>(sm + OFF_X);
    float* cs = reinterpret_cast<float*>(sm + OFF_CS);
    float4* pst = reinterpret_cast<float4*>(sm + OFF_P);

    if (tid == 0) {
        s_abort = 0;
        s_max_tiles = 1;
        ring_init(ring);
        fence_barrier_init();
    }
    for (int i = tid; i < (int)(2 * sizeof(PassSlot) / 4); i += STHREADS) reinterpret_cast<int*>(ring.slot)[i] = 0;
    // both operands start as zeros: columns past H and rows of hidden units past H stay that way
    for (int i = tid; i < (OFF_X - OFF_U) / 16; i += STHREADS) reinterpret_cast<float4*>(sm + OFF_U)[i] = make_float4(0.f, 0.f, 0.f, 0.f);
    __syncthreads();
    // resident weight slice
    for (int idx = tid; idx < H * SBJ; idx += STHREADS) {
        const int jj = idx & (SBJ - 1), k = idx >> 5;
        if (j0 + jj < H) {
            const float4 u = __ldg(&a.Ut4[(size_t)k * H + j0 + jj]);
            us[(0 * SBJ + jj) * LDF + k] = u.x;
            us[(1 * SBJ + jj) * LDF + k] = u.y;
            us[(2 * SBJ + jj) * LDF + k] = u.z;
            us[(3 * SBJ + jj) * LDF + k] = u.w;
        }
    }
    __syncthreads();
    volatile int* abort = &s_abort;

    const int n_levels = a.meta[META_N_LEVELS];
    const bool bad_forest = a.meta[META_ERROR] != 0 || a.meta[META_UNFINISHED] != 0;
    const int n_leaves = n_levels > 0 ? a.level_ptr[1] : 0;
    bool alive = !bad_forest;

    // Only as many tile groups as the largest level has tiles take part; the others leave before the first
    // barrier, which therefore counts the participating CTAs only.
    {
        int mt = 1;
        for (int l = 1 + tid; l < n_levels; l += STHREADS) {
            int llo, lhi;
            checked_level(a.level_ptr, l, a.n_nodes, a.meta, a.debug, llo, lhi);
            const int ln = lhi - llo, nt = tile_nodes(ln, FNT_RULE, n_grp);
            mt = max(mt, (ln + nt - 1) / nt);
        }
        if (mt > 1) atomicMax(&s_max_tiles, mt);
    }
    __syncthreads();
    const int active_grp = min(n_grp, s_max_tiles);
    const unsigned active_ctas = (unsigned)(active_grp * a.n_slices);
    if (grp >= active_grp) alive = false;

    if (warp >= MAIN_WARPS) {
        // ================= description warps =================
        if (alive) {
            DescribeArgs d{a.child_ptr, a.child_idx, a.level_ptr, a.perm, nullptr, 1, n_levels, grp, n_grp, active_grp, FNT_RULE,
                           a.meta, a.n_nodes, a.n_edges, a.debug, nullptr, nullptr, 0, n_leaves};
            describe_passes(d, ring, FET, abort, tid - MAIN_THREADS, [&](const PassSlot& S, int m, int tcount, int tm) {
                // the tile's input projection for this CTA's hidden units (parity selects the buffer)
                float4* dst = pst + (tcount & 1) * (FNT * SBJ);
                for (int task = tm; task < m * SBJ; task += META_THREADS) {
                    const int r = task >> 5, jj = task & 31;
                    if (j0 + jj < H) cp_async16(smem_u32(dst + r * SBJ + jj), a.P4 + (size_t)S.prow[r] * H + j0 + jj);
                    else dst[r * SBJ + jj] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
            });
        }
    } else {
        // ================= arithmetic warps =================
        auto stamp = [&](int level, int s, bool first) {
            if (a.trace && first && blockIdx.x == 0 && tid == 0 && (long long)level * 8 + s < a.trace_cap)
                a.trace[level * 8 + s] = global_ns();
        };
        // register tile of the products: outputs n = 32 gate + (lane & 7) + 8 i, edges e = e_base + 4 i'
        const int gate = warp & 3;
        const int n_base = gate * SBJ + (lane & 7);
        const int e_base = (lane >> 3) + 8 * (warp >> 2);
        const float4* us4 = reinterpret_cast<const float4*>(us);
        const float4* hk4 = reinterpret_cast<const float4*>(hk);
        int k = 0, tcount = 0;
        for (int level = 1; level < n_levels && alive; ++level) {
            int lo, hi;
            checked_level(a.level_ptr, level, a.n_nodes, a.meta, a.debug, lo, hi);
            const int nt = tile_nodes(hi - lo, FNT_RULE, n_grp);
            const int tiles = (hi - lo + nt - 1) / nt;
            stamp(level, 0, true);
            for (int tile = grp; tile < tiles && alive; tile += active_grp, ++tcount) {
                const bool first = tile == grp;
                float zi[2], zo[2], zu[2], sfc[2];  // running sums of this thread's (row, hidden unit) pairs
#pragma unroll
                for (int i = 0; i < 2; ++i) zi[i] = zo[i] = zu[i] = sfc[i] = 0.f;
                bool last = false;
                while (!last) {
                    const int s = k & 1;
                    const bool good = mbar_wait_warp(smem_u32(&ring.bar_full[s]), (uint32_t)((k >> 1) & 1), abort);
                    if (!good) *abort = 1;
                    const PassSlot& S = ring.slot[s];
                    const int m = S.m, ne = S.ne, et0 = S.et0;
                    const int nc = good ? min(FET, ne - et0) : 0;
                    last = !good || et0 + FET >= ne;
                    stamp(level, 1, first && et0 == 0);
                    // ---- gather: fp32 child rows and c slices ----
                    for (int e = warp; e < nc; e += MAIN_WARPS) {
                        const float* hrow = a.h + (int64_t)S.ek_id[e] * a.ldh;
                        for (int c4 = lane; c4 < kq; c4 += 32) {
                            if (a.vec_ok && 4 * c4 + 4 <= H) cp_async16(smem_u32(hk + e * LDF + 4 * c4), hrow + 4 * c4);
                            else *reinterpret_cast<float4*>(hk + e * LDF + 4 * c4) = load_row4(hrow, 4 * c4, H, a.vec_ok);
                        }
                    }
                    for (int task = tid; task < nc * (SBJ / 4); task += MAIN_THREADS) {
                        const int e = task >> 3, q = task & 7;
                        const float* crow = a.c + (int64_t)S.ek_id[e] * a.ldh;
                        if (a.vec_ok && j0 + 4 * q + 4 <= H) cp_async16(smem_u32(cs + e * CS_LD + 4 * q), crow + j0 + 4 * q);
                        else *reinterpret_cast<float4*>(cs + e * CS_LD + 4 * q) = load_row4(crow, j0 + 4 * q, H, a.vec_ok);
                    }
                    cp_async_wait_all();
                    if (named_bar_any(BAR_MAIN, MAIN_THREADS, !good || s_abort != 0)) { alive = false; break; }  // one verdict for all warps
                    stamp(level, 2, first && et0 == 0);
                    // ---- products: 2 edges x 4 outputs per thread, K ascending ----
                    float acc[2][4];
#pragma unroll
                    for (int ie = 0; ie < 2; ++ie)
#pragma unroll
                        for (int in = 0; in < 4; ++in) acc[ie][in] = 0.f;
                    if (e_base < nc) {  // rows past the pass's edges hold older rows: finite, and never read back
#pragma unroll 2
                        for (int k4 = 0; k4 < kq; ++k4) {
                            float4 hv[2], uv[4];
#pragma unroll
                            for (int ie = 0; ie < 2; ++ie) hv[ie] = hk4[(e_base + 4 * ie) * LDK + k4];
#pragma unroll
                            for (int in = 0; in < 4; ++in) uv[in] = us4[(n_base + 8 * in) * LDK + k4];
#pragma unroll
                            for (int ie = 0; ie < 2; ++ie)
#pragma unroll
                                for (int in = 0; in < 4; ++in) {
                                    acc[ie][in] = fmaf(hv[ie].x, uv[in].x, acc[ie][in]);
                                    acc[ie][in] = fmaf(hv[ie].y, uv[in].y, acc[ie][in]);
                                    acc[ie][in] = fmaf(hv[ie].z, uv[in].z, acc[ie][in]);
                                    acc[ie][in] = fmaf(hv[ie].w, uv[in].w, acc[ie][in]);
                                }
                        }
                    }
                    stamp(level, 4, first && et0 == 0);
                    // ---- hand-over: i, o, u shares as they are, forget columns as f_jk c_k ----
#pragma unroll
                    for (int ie = 0; ie < 2; ++ie) {
                        const int e = e_base + 4 * ie;
                        if (e >= nc) continue;
#pragma unroll
                        for (int in = 0; in < 4; ++in) {
                            const int jj = (lane & 7) + 8 * in;
                            float val = acc[ie][in];
                            if (gate == 3) {
                                const float pf = pst[(tcount & 1) * (FNT * SBJ) + S.ep[e] * SBJ + jj].w;
                                val = sigmoid_acc(pf + val) * cs[e * CS_LD + jj];
                            }
                            xch[e * XLD + gate * SBJ + jj] = val;
                        }
                    }
                    named_bar(BAR_MAIN, MAIN_THREADS);
                    stamp(level, 5, first && et0 == 0);
                    // ---- cell arithmetic: one thread per (row, hidden unit) ----
#pragma unroll
                    for (int i = 0; i < 2; ++i) {
                        const int r = warp + MAIN_WARPS * i;
                        if (r >= m) continue;
                        const int ea = max(S.eoff[r], et0), eb = min(S.eoff[r + 1], et0 + FET);
                        for (int e = ea; e < eb; ++e) {  // CSR order
                            const float* src = xch + (e - et0) * XLD + lane;
                            zi[i] += src[0];
                            zo[i] += src[SBJ];
                            zu[i] += src[2 * SBJ];
                            sfc[i] += src[3 * SBJ];
                        }
                        if (last && j0 + lane < H && S.nodes[r] >= 0) {
                            const float4 p = pst[(tcount & 1) * (FNT * SBJ) + r * SBJ + lane];
                            const float cc = fmaf(sigmoid_acc(zi[i] + p.x), tanhf(zu[i] + p.z), sfc[i]);
                            const int64_t row = (int64_t)S.nodes[r] * a.ldh;
                            a.c[row + j0 + lane] = cc;
                            a.h[row + j0 + lane] = sigmoid_acc(zo[i] + p.y) * tanhf(cc);
                        }
                    }
                    named_bar(BAR_MAIN, MAIN_THREADS);  // exchange buffer, child rows and slot are free again
                    if (tid == 0) mbar_arrive(smem_u32(&ring.bar_empty[s]));
                    stamp(level, 6, first && last);
                    ++k;
                }
            }
            if (!alive) break;
            if (level + 1 < n_levels) {
                if (!main_grid_barrier(a.meta, &a.meta[META_BARRIER], (unsigned)level * active_ctas, a.timeout_ns, abort, tid)) alive = false;
            }
            stamp(level, 7, true);
        }
    }

    __syncthreads();
    if (s_abort && tid == 0) atomicExch(&a.meta[META_TIMEOUT], 1);
}

}  // namespace

bool small_levels_f32_supported(int32_t H) { return H <= FMAX_H; }

jdb_status small_levels_f32_enqueue(const ForwardArgs& fa, int n_internal_bound, uint64_t timeout_ns, cudaStream_t st) {
    const int H = fa.H;
    if (!small_levels_f32_supported(H)) return JDB_ERR_UNSUPPORTED;
    DevInfo* di = dev_info();
    if (!di) return JDB_ERR_CUDA;
    if (!(di->attr_mask & ATTR_SMALL_F32)) {
        JDB_CUDA_TRY(cudaFuncSetAttribute(small_levels_f32_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, F32_SMEM));
        int per_sm = 0;
        JDB_CUDA_TRY(cudaOccupancyMaxActiveBlocksPerMultiprocessor(&per_sm, small_levels_f32_kernel, STHREADS, F32_SMEM));
        if (per_sm < 1) return JDB_ERR_UNSUPPORTED;
        di->attr_mask |= ATTR_SMALL_F32;
    }
    F32Args a{};
    a.child_ptr = fa.child_ptr; a.child_idx = fa.child_idx; a.level_ptr = fa.level_ptr; a.perm = fa.perm;
    a.meta = fa.meta; a.H = H;
    a.n_nodes = fa.n_nodes; a.n_edges = fa.n_edges; a.debug = fa.debug;
    a.n_slices = (H + SBJ - 1) / SBJ;
    a.Ut4 = (const float4*)fa.Ut;
    a.P4 = (const float4*)fa.P;
    a.h = fa.h; a.c = fa.c; a.ldh = fa.ldh;
    a.vec_ok = (fa.ldh % 4 == 0) && (((uintptr_t)fa.h & 15) == 0) && (((uintptr_t)fa.c & 15) == 0);
    a.timeout_ns = timeout_ns;
    a.trace = fa.trace;
    a.trace_cap = fa.trace_cap;

    int groups = di->n_sm / a.n_slices;  // one CTA per SM
    const int max_tiles = ceil_div(n_internal_bound > 0 ? n_internal_bound : 1, 4);
    if (groups > max_tiles) groups = max_tiles;
    if (groups < 1) return JDB_ERR_UNSUPPORTED;
    void* params[] = {&a};
    JDB_CUDA_TRY(cudaLaunchCooperativeKernel((const void*)small_levels_f32_kernel, dim3(groups * a.n_slices), dim3(STHREADS),
                                             params, F32_SMEM, st));
    return JDB_OK;
}

}  // namespace jdb
