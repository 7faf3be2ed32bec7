// Requests that arrive one after the other (the serving case of Section 2: a batching analysis that has to run before
// execution suits requests arriving irregularly only if it is cheap and does not wait for a full batch).  Every request
// is a forest of its own; it gets the next of a few slots, each with its own stream and its own part of the caller's
// device scratch, so that the copies and the analysis of a new request run while earlier requests execute.  Host code
// only: the kernels are those of jdb_treelstm_forward_host.
#include <new>
#include <vector>

#include "common.cuh"

struct jdb_online {
    int32_t slots, max_nodes, max_edges, D, H, x_dtype;
    jdb_opts opts;
    const void* packed;
    char* ws;
    size_t slot_bytes;
    std::vector<cudaStream_t> streams;
    std::vector<int32_t*> meta;        // per slot: status words of the request in flight (null: none, or an empty forest)
    std::vector<int64_t> in_flight;    // per slot: ticket in flight, -1 = free
    std::vector<signed char> status;   // per ticket: -1 pending, else its jdb_status
    std::vector<int32_t> levels;       // per ticket: level count once known
};

using namespace jdb;

namespace {

// waits for the request in `slot` and files its status under its ticket
jdb_status finish_slot(jdb_online* o, int slot) {
    const int64_t t = o->in_flight[slot];
    if (t < 0) return JDB_OK;
    int32_t n_levels = 0;
    JDB_CUDA_TRY(cudaStreamSynchronize(o->streams[slot]));
    const jdb_status s = forward_host_finish(o->meta[slot], &n_levels, o->streams[slot]);
    o->status[(size_t)t] = (signed char)s;
    o->levels[(size_t)t] = n_levels;
    o->in_flight[slot] = -1;
    o->meta[slot] = nullptr;
    return JDB_OK;
}

}  // namespace

extern "C" {

size_t jdb_online_workspace_bytes(int32_t slots, int32_t max_nodes, int32_t max_edges, int32_t D, int32_t H, int32_t precision,
                                  int32_t x_dtype) {
    if (slots < 1 || max_nodes < 0 || max_edges < 0 || D <= 0 || H <= 0) return 0;
    return (size_t)slots * align_up(jdb_forward_host_workspace_bytes(max_nodes, max_edges, D, H, precision, x_dtype), 256);
}

jdb_status jdb_online_create(jdb_online** out, int32_t slots, int32_t max_nodes, int32_t max_edges, const void* packed, int32_t D,
                             int32_t H, const jdb_opts* opts, int32_t x_dtype, void* dev_ws, size_t dev_ws_bytes) {
    if (!out) return JDB_ERR_INVALID_ARG;
    *out = nullptr;
    if (slots < 1 || slots > 16 || max_nodes < 1 || max_edges < 0 || !packed || !opts || D <= 0 || H <= 0) return JDB_ERR_INVALID_ARG;
    if (x_dtype != JDB_FP32 && x_dtype != JDB_BF16) return JDB_ERR_INVALID_ARG;
    if (!dev_ws || ((uintptr_t)dev_ws & 255) != 0) return JDB_ERR_INVALID_ARG;
    if (dev_ws_bytes < jdb_online_workspace_bytes(slots, max_nodes, max_edges, D, H, opts->precision, x_dtype)) return JDB_ERR_WORKSPACE;
    jdb_online* o = new (std::nothrow) jdb_online();
    if (!o) return JDB_ERR_INVALID_ARG;
    o->slots = slots; o->max_nodes = max_nodes; o->max_edges = max_edges; o->D = D; o->H = H; o->x_dtype = x_dtype;
    o->opts = *opts;
    o->opts.ev_begin = o->opts.ev_xproj_done = o->opts.ev_levels_done = nullptr;   // per-call hooks make no sense across requests
    o->opts.trace = nullptr;
    o->packed = packed;
    o->ws = (char*)dev_ws;
    o->slot_bytes = align_up(jdb_forward_host_workspace_bytes(max_nodes, max_edges, D, H, opts->precision, x_dtype), 256);
    o->meta.assign(slots, nullptr);
    o->in_flight.assign(slots, -1);
    for (int i = 0; i < slots; ++i) {
        cudaStream_t st = nullptr;
        cudaError_t e = cudaStreamCreateWithFlags(&st, cudaStreamNonBlocking);
        if (e != cudaSuccess) {
            set_last_cuda_error(e);
            for (cudaStream_t s : o->streams) cudaStreamDestroy(s);
            delete o;
            return JDB_ERR_CUDA;
        }
        o->streams.push_back(st);
    }
    *out = o;
    return JDB_OK;
}

jdb_status jdb_online_submit(jdb_online* o, const int32_t* child_ptr, const int32_t* child_idx, int32_t n_nodes, int32_t n_edges,
                             const void* x, float* h, float* c, int64_t* ticket) {
    if (!o || !ticket) return JDB_ERR_INVALID_ARG;
    *ticket = -1;
    if (n_nodes < 0 || n_edges < 0) return JDB_ERR_INVALID_ARG;
    if (n_nodes > o->max_nodes || n_edges > o->max_edges) return JDB_ERR_WORKSPACE;
    const int64_t t = (int64_t)o->status.size();
    const int slot = (int)(t % o->slots);
    jdb_status s = finish_slot(o, slot);   // the slot's earlier request, if nobody waited for it yet
    if (s != JDB_OK) return s;
    int32_t* meta = nullptr;
    s = forward_host_enqueue(child_ptr, child_idx, n_nodes, n_edges, x, o->x_dtype, o->packed, o->D, o->H, h, c, &o->opts,
                             o->ws + (size_t)slot * o->slot_bytes, o->slot_bytes, &meta, o->streams[slot]);
    if (s != JDB_OK) {
        // whatever part was enqueued must not outlive this call's view of the slot
        cudaStreamSynchronize(o->streams[slot]);
        return s;
    }
    o->status.push_back(-1);
    o->levels.push_back(0);
    o->in_flight[slot] = t;
    o->meta[slot] = meta;
    *ticket = t;
    return JDB_OK;
}

jdb_status jdb_online_wait(jdb_online* o, int64_t ticket, int32_t* n_levels_out) {
    if (n_levels_out) *n_levels_out = 0;
    if (!o || ticket < 0 || ticket >= (int64_t)o->status.size()) return JDB_ERR_INVALID_ARG;
    if (o->status[(size_t)ticket] < 0) {
        const int slot = (int)(ticket % o->slots);
        if (o->in_flight[slot] != ticket) return JDB_ERR_INVALID_ARG;   // cannot happen: a pending ticket owns its slot
        const jdb_status s = finish_slot(o, slot);
        if (s != JDB_OK) return s;
    }
    if (n_levels_out) *n_levels_out = o->levels[(size_t)ticket];
    return (jdb_status)o->status[(size_t)ticket];
}

jdb_status jdb_online_destroy(jdb_online* o) {
    if (!o) return JDB_OK;
    jdb_status r = JDB_OK;
    for (int i = 0; i < o->slots; ++i) {
        if (cudaStreamSynchronize(o->streams[i]) != cudaSuccess) r = JDB_ERR_CUDA;
        cudaStreamDestroy(o->streams[i]);
    }
    delete o;
    return r;
}

}  // extern "C"
