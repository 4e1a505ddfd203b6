// The C ABI: argument checks, device-state layout and the per-batch kernel sequence.
#include <atomic>
#include <cmath>
#include <cstdarg>
#include <cstdio>
#include <cstring>
#include <new>

#include "gs_internal.h"

struct gs_graph {
    int64_t num_nodes, num_edges;
    const int64_t* d_indptr;
    const int32_t* d_indices;
    const void* d_features;
    gs_dtype dtype;
    int32_t feat_dim;
    int64_t feat_ld;
    int32_t elem_bytes;
    int32_t gather_blocks_per_sm;   // grid of gs_gather_features; 0 = the library's default
};

struct gs_cache {
    const gs_graph* graph;
    int32_t L, W, pitch, shared, num_caches;
    int32_t fanouts[GS_MAX_HOPS];
    uint64_t seed;
    char* d_storage;
    int32_t* d_hdr;
    unsigned long long* d_table;
    int32_t* d_slots;
    size_t slot_bytes;        // all caches
    uint32_t serial;          // batches run; the relabel stamp is derived from it
    uint32_t shard_stamp;     // stamp of the sharded batch in progress (gs_shard_extend)
    int32_t shard_seeds;      // its number of seeds
    float lambda_otf, lambda_full;
    int32_t hub_degree;
    int32_t theta;            // split cache: nodes with degree <= theta have no row (-1: every node has one)
    int64_t rows;             // cache rows per cache (num_nodes, or the dense nodes of a split cache)
    int32_t* d_row_index;     // split cache only
    int32_t dedup;            // DedupMethod of gs_sample_batch
    int32_t* h_pinned;        // pinned staging for counts
    // optional device timing of the kernel groups (gs_cache_profile_begin / _end)
    cudaEvent_t* prof_events;
    int32_t prof_cap, prof_used;   // in batches
};

constexpr int PROF_GROUPS = 4;               // row counts | scan | finish or fused refresh+pick | relabel
constexpr int PROF_EVENTS_PER_STEP = PROF_GROUPS + 1;

namespace gs {

static thread_local char g_err[512] = "";
static std::atomic<long long> g_launches{0};

void count_launches(int n) { g_launches.fetch_add(n, std::memory_order_relaxed); }

static std::atomic<int> g_sm_count[64];     // per device ordinal, 0 = not looked up yet
static std::atomic<int> g_grid_cap{0};      // test knob: 0 = grids as designed

int64_t sm_count() {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return 148;
    int n = g_sm_count[dev].load(std::memory_order_relaxed);
    if (n <= 0) {
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        g_sm_count[dev].store(n, std::memory_order_relaxed);
    }
    return n;
}

int64_t limit_grid(int64_t blocks) {
    const int cap = g_grid_cap.load(std::memory_order_relaxed);
    if (cap > 0 && blocks > cap) blocks = cap;
    return blocks < 1 ? 1 : blocks;
}

static gs_status fail(gs_status code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

gs_status set_error(gs_status code, const char* fmt, ...) {
    va_list ap;
    va_start(ap, fmt);
    vsnprintf(g_err, sizeof(g_err), fmt, ap);
    va_end(ap);
    return code;
}

static gs_status cuda_fail(cudaError_t e, const char* what) {
    return fail(GS_ERR_CUDA, "%s: %s", what, cudaGetErrorString(e));
}

#define GS_CUDA(call)                                          \
    do {                                                       \
        cudaError_t e__ = (call);                              \
        if (e__ != cudaSuccess) return cuda_fail(e__, #call);  \
    } while (0)

static bool aligned(const void* p, size_t a) { return ((uintptr_t)p % a) == 0; }

static int32_t pitch_for(int32_t W) { return (W + 7) / 8 * 8; }

static gs_status check_shape(const gs_graph* g, int32_t num_hops, int32_t cache_width) {
    if (!g) return fail(GS_ERR_ARG, "graph is NULL");
    if (num_hops < 1 || num_hops > GS_MAX_HOPS) return fail(GS_ERR_ARG, "num_hops %d outside [1, %d]", num_hops, GS_MAX_HOPS);
    if (cache_width < 1 || cache_width > GS_MAX_CACHE_WIDTH)
        return fail(GS_ERR_ARG, "cache_width %d outside [1, %d]", cache_width, GS_MAX_CACHE_WIDTH);
    return GS_OK;
}

static size_t table_bytes(const gs_graph* g) { return align_up((size_t)g->num_nodes * 8, 256); }
static size_t slots_bytes(const gs_graph* g, int32_t caches, int32_t W) {
    return align_up((size_t)caches * (size_t)g->num_nodes * (size_t)pitch_for(W) * 4, 256);
}

static uint32_t key_word(uint32_t purpose, uint32_t tag) { return (purpose << 8) | tag; }

static StepParams step_params(const gs_cache* c, int32_t layer, uint32_t step) {
    StepParams P{};
    const gs_graph* g = c->graph;
    P.g = GraphView{g->d_indptr, g->d_indices, g->num_nodes};
    const int32_t ci = c->shared ? 0 : layer;
    P.slots = c->d_slots + (size_t)ci * (size_t)c->rows * c->pitch;
    P.row_index = c->d_row_index;
    P.theta = c->theta;
    P.word_fetch = key_word(4, (uint32_t)layer);
    P.pitch = c->pitch;
    P.W = c->W;
    P.f = c->fanouts[layer];
    P.step = step;
    P.key0 = (uint32_t)(c->seed & 0xFFFFFFFFu);
    P.key1 = (uint32_t)(c->seed >> 32);
    for (int i = 0; i < 10; ++i) {
        P.rk[2 * i] = P.key0 + (uint32_t)i * 0x9E3779B9u;
        P.rk[2 * i + 1] = P.key1 + (uint32_t)i * 0xBB67AE85u;
    }
    const uint32_t ctag = c->shared ? 0xFFu : (uint32_t)layer;
    P.word_fill = key_word(1, ctag);
    P.word_evict = key_word(2, ctag);
    P.word_pick = key_word(3, (uint32_t)layer);
    P.table = c->d_table;
    P.status = c->d_hdr + HDR_STATUS;
    P.stats = c->d_hdr + HDR_STAT_SLOW;
    P.lambda_otf = c->lambda_otf;
    P.lambda_full = c->lambda_full;
    P.hub_degree = c->hub_degree;
    return P;
}

}  // namespace gs

using namespace gs;

extern "C" {

const char* gs_last_error(void) { return g_err; }
int32_t gs_stats_word_offset(void) { return HDR_STAT_SLOW; }
int64_t gs_kernel_launches(void) { return (int64_t)g_launches.load(); }

gs_status gs_debug_set_grid_cap(int32_t max_blocks) {
    if (max_blocks < 0) return fail(GS_ERR_ARG, "max_blocks is negative");
    g_grid_cap.store(max_blocks, std::memory_order_relaxed);
    return GS_OK;
}

gs_status gs_graph_create(int64_t num_nodes, int64_t num_edges, const int64_t* d_indptr, const int32_t* d_indices,
                          const void* d_features, gs_dtype dtype, int32_t feat_dim, int64_t feat_ld, gs_graph** out) {
    if (!out) return fail(GS_ERR_ARG, "out is NULL");
    *out = nullptr;
    if (num_nodes < 1 || num_nodes >= ((int64_t)1 << 31)) return fail(GS_ERR_ARG, "num_nodes %lld outside [1, 2^31)", (long long)num_nodes);
    if (num_edges < 0) return fail(GS_ERR_ARG, "num_edges is negative");
    if (!d_indptr) return fail(GS_ERR_ARG, "d_indptr is NULL");
    if (!d_indices && num_edges > 0) return fail(GS_ERR_ARG, "d_indices is NULL");
    if (!aligned(d_indptr, 8)) return fail(GS_ERR_ALIGN, "d_indptr must be 8-byte aligned");
    if (!aligned(d_indices, 4)) return fail(GS_ERR_ALIGN, "d_indices must be 4-byte aligned");
    if (dtype != GS_F32 && dtype != GS_BF16) return fail(GS_ERR_ARG, "unknown dtype %d", (int)dtype);
    const int32_t eb = dtype == GS_F32 ? 4 : 2;
    if (d_features) {
        if (feat_dim < 1) return fail(GS_ERR_ARG, "feat_dim must be >= 1");
        if (feat_ld < feat_dim) return fail(GS_ERR_ARG, "feat_ld %lld < feat_dim %d", (long long)feat_ld, feat_dim);
        if (!aligned(d_features, (size_t)eb)) return fail(GS_ERR_ALIGN, "d_features must be aligned to its element size");
    }
    gs_graph* g = new (std::nothrow) gs_graph{num_nodes, num_edges, d_indptr, d_indices, d_features, dtype, feat_dim, feat_ld, eb, 0};
    if (!g) return fail(GS_ERR_ARG, "out of host memory");
    *out = g;
    return GS_OK;
}

void gs_graph_destroy(gs_graph* g) { delete g; }

gs_status gs_graph_set_gather_grid(gs_graph* g, int32_t blocks_per_sm) {
    if (!g) return fail(GS_ERR_ARG, "graph is NULL");
    if (blocks_per_sm < -1 || blocks_per_sm > 4096) return fail(GS_ERR_ARG, "blocks_per_sm outside [-1, 4096]");
    g->gather_blocks_per_sm = blocks_per_sm;
    return GS_OK;
}

gs_status gs_gather_status(void* stream) {
    int flag = 0;
    GS_CUDA(gather_gave_up((cudaStream_t)stream, &flag));
    if (flag) return fail(GS_ERR_CUDA, "a feature gather gave up waiting for a bulk copy");
    return GS_OK;
}

gs_status gs_graph_validate(const gs_graph* g, void* stream, int64_t* h_first_bad_row) {
    if (!g || !h_first_bad_row) return fail(GS_ERR_ARG, "NULL argument");
    GS_CUDA(launch_validate_graph(GraphView{g->d_indptr, g->d_indices, g->num_nodes}, g->num_edges, h_first_bad_row,
                                  (cudaStream_t)stream));
    if (*h_first_bad_row >= 0)
        return fail(GS_ERR_ARG, "CSR row %lld breaks the graph contract (offsets, id range, or ids not strictly ascending)",
                    (long long)*h_first_bad_row);
    return GS_OK;
}

gs_status gs_graph_count_dense(const gs_graph* g, int32_t theta, void* stream, int64_t* h_dense_rows) {
    if (!g || !h_dense_rows) return fail(GS_ERR_ARG, "NULL argument");
    if (theta < 0) return fail(GS_ERR_ARG, "theta must be >= 0");
    GS_CUDA(launch_count_dense(GraphView{g->d_indptr, g->d_indices, g->num_nodes}, theta, h_dense_rows, (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_cache_bytes(const gs_graph* g, int32_t num_hops, int32_t cache_width, int32_t shared, size_t* bytes) {
    if (!bytes) return fail(GS_ERR_ARG, "bytes is NULL");
    gs_status st = check_shape(g, num_hops, cache_width);
    if (st != GS_OK) return st;
    *bytes = HDR_BYTES + table_bytes(g) + slots_bytes(g, shared ? 1 : num_hops, cache_width);
    return GS_OK;
}

static gs_status check_fanouts(int32_t num_hops, const int32_t* fanouts, int32_t limit) {
    if (!fanouts) return fail(GS_ERR_ARG, "fanouts is NULL");
    for (int l = 0; l < num_hops; ++l)
        if (fanouts[l] < 1 || fanouts[l] > limit) return fail(GS_ERR_ARG, "fanouts[%d] = %d outside [1, %d]", l, fanouts[l], limit);
    return GS_OK;
}

gs_status gs_workspace_bytes(const gs_graph* g, int32_t num_hops, const int32_t* fanouts, int32_t max_seeds, size_t* bytes) {
    if (!bytes) return fail(GS_ERR_ARG, "bytes is NULL");
    gs_status st = check_shape(g, num_hops, 1);
    if (st != GS_OK) return st;
    st = check_fanouts(num_hops, fanouts, GS_MAX_CACHE_WIDTH);
    if (st != GS_OK) return st;
    if (max_seeds < 1) return fail(GS_ERR_ARG, "max_seeds must be >= 1");
    const Bounds b = make_bounds(g->num_nodes, num_hops, fanouts, max_seeds);
    for (int k = 0; k < num_hops; ++k)
        if (b.nb[k] + b.mb[k] >= ((int64_t)1 << 31)) return fail(GS_ERR_ARG, "batch too large: positions would exceed 2^31");
    *bytes = make_layout(b, g->num_edges).total;
    return GS_OK;
}

static size_t row_index_bytes(const gs_graph* g) { return align_up((size_t)g->num_nodes * 4, 256); }

gs_status gs_cache_bytes_split(const gs_graph* g, int32_t num_hops, int32_t cache_width, int32_t shared,
                               int64_t dense_rows, size_t* bytes) {
    if (!bytes) return fail(GS_ERR_ARG, "bytes is NULL");
    gs_status st = check_shape(g, num_hops, cache_width);
    if (st != GS_OK) return st;
    if (dense_rows < 0 || dense_rows > g->num_nodes) return fail(GS_ERR_ARG, "dense_rows outside [0, num_nodes]");
    const size_t rows = (size_t)(dense_rows > 0 ? dense_rows : 1);
    *bytes = HDR_BYTES + table_bytes(g) + row_index_bytes(g) +
             align_up((size_t)(shared ? 1 : num_hops) * rows * (size_t)pitch_for(cache_width) * 4, 256);
    return GS_OK;
}

// Refreshes r slots of every cached row (all caches) with the keys of `step`: the fused per-node
// kernels over the node range instead of a frontier.  init = 1 writes whole rows (the pre-sample).
// The relabel table is idle between batches and serves as the hub storage of these launches (the
// hub degree is raised until the hubs it can produce fit there); it is reset afterwards, which is
// the state every batch expects of entries it has not stamped.
static cudaError_t refresh_every_row(gs_cache* c, int32_t r, uint32_t step, int init, cudaStream_t s) {
    const gs_graph* g = c->graph;
    const size_t table_room = (size_t)g->num_nodes * 8;
    int64_t hub_degree0 = c->hub_degree < HUB_MIN_DEGREE ? HUB_MIN_DEGREE : c->hub_degree;
    int64_t cap0 = 0, items0 = 0;
    size_t o_entry = 0, o_state = 0, o_items = 0, o_cand = 0;
    for (int tries = 0; tries < 40; ++tries, hub_degree0 *= 2) {
        cap0 = g->num_edges / hub_degree0 + 1;
        if (cap0 > g->num_nodes) cap0 = g->num_nodes;
        items0 = g->num_edges / (4 * (int64_t)HUB_CHUNK_QUADS) + cap0 + 1;
        o_entry = 0;
        o_state = align_up(o_entry + (size_t)cap0 * 8, 256);
        o_items = align_up(o_state + (size_t)cap0 * 8, 256);
        o_cand = align_up(o_items + (size_t)items0 * 4, 256);
        if (o_cand + (size_t)cap0 * HUB_CAND_CAP * 8 <= table_room) break;
        cap0 = 0;
    }
    cudaError_t e = cudaSuccess;
    for (int ci = 0; ci < c->num_caches; ++ci) {
        StepParams P = step_params(c, ci, step);
        P.r = r;
        P.frontier = nullptr;
        P.d_n = nullptr;
        P.n_host = (int32_t)g->num_nodes;
        P.d_refresh_from = nullptr;
        P.do_pick = 0;
        P.init_rows = init;
        char* hub_base = (char*)c->d_table;
        P.hub_entry = (int2*)(hub_base + o_entry);
        P.hub_state = (int2*)(hub_base + o_state);
        P.hub_items = (int32_t*)(hub_base + o_items);
        P.hub_cand = (unsigned long long*)(hub_base + o_cand);
        P.hub_counter = (unsigned long long*)(c->d_hdr + HDR_HUB64 + 2 * ci);
        P.hub_cap = (int32_t)cap0;          // 0: the table is too small, every node is done by one warp
        P.item_cap = (int32_t)items0;
        P.hub_degree = cap0 > 0 ? (int32_t)(hub_degree0 > 0x7FFFFFFF ? 0x7FFFFFFF : hub_degree0) : 0x7FFFFFFF;
        P.work_counter = c->d_hdr + HDR_WORK + ci;
        P.work_counter2 = c->d_hdr + HDR_WORK2 + ci;
        e = launch_refresh_pick(P, g->num_nodes, s);
        if (e != cudaSuccess) return e;
    }
    return cudaMemsetAsync(c->d_table, 0xFF, (size_t)g->num_nodes * 8, s);
}

static gs_status cache_init_impl(const gs_graph* g, int32_t num_hops, const int32_t* fanouts, int32_t cache_width,
                                 uint64_t seed, int32_t shared, int32_t theta, int64_t dense_rows,
                                 void* d_cache_storage, size_t cache_bytes, void* stream, gs_cache** out) {
    if (!out) return fail(GS_ERR_ARG, "out is NULL");
    *out = nullptr;
    gs_status st = check_shape(g, num_hops, cache_width);
    if (st != GS_OK) return st;
    st = check_fanouts(num_hops, fanouts, cache_width);
    if (st != GS_OK) return st;
    if (!d_cache_storage) return fail(GS_ERR_ARG, "d_cache_storage is NULL");
    if (!aligned(d_cache_storage, 256)) return fail(GS_ERR_ALIGN, "d_cache_storage must be 256-byte aligned");
    const bool split_cache = theta >= 0;
    if (split_cache && (theta < cache_width || theta > SMALL_DEGREE))
        return fail(GS_ERR_ARG, "theta %d outside [cache_width, %d]", theta, SMALL_DEGREE);
    size_t need = 0;
    if (split_cache) st = gs_cache_bytes_split(g, num_hops, cache_width, shared, dense_rows, &need);
    else st = gs_cache_bytes(g, num_hops, cache_width, shared, &need);
    if (st != GS_OK) return st;
    if (cache_bytes < need) return fail(GS_ERR_WORKSPACE, "cache storage has %zu bytes, %zu needed", cache_bytes, need);

    // the built-in scratch array of gs_sample_batch_noalloc comes into being on this device now, not in a later batch
    st = prepare_noalloc_scratch();
    if (st != GS_OK) return st;

    gs_cache* c = new (std::nothrow) gs_cache{};
    if (!c) return fail(GS_ERR_ARG, "out of host memory");
    c->graph = g;
    c->L = num_hops;
    c->W = cache_width;
    c->pitch = pitch_for(cache_width);
    c->shared = shared ? 1 : 0;
    c->num_caches = shared ? 1 : num_hops;
    memcpy(c->fanouts, fanouts, (size_t)num_hops * sizeof(int32_t));
    c->seed = seed;
    c->d_storage = (char*)d_cache_storage;
    c->d_hdr = (int32_t*)c->d_storage;
    c->d_table = (unsigned long long*)(c->d_storage + HDR_BYTES);
    c->theta = split_cache ? theta : -1;
    c->rows = split_cache ? (dense_rows > 0 ? dense_rows : 1) : g->num_nodes;
    c->d_row_index = split_cache ? (int32_t*)(c->d_storage + HDR_BYTES + table_bytes(g)) : nullptr;
    c->d_slots = (int32_t*)(c->d_storage + HDR_BYTES + table_bytes(g) + (split_cache ? row_index_bytes(g) : 0));
    c->slot_bytes = (size_t)c->num_caches * (size_t)c->rows * (size_t)c->pitch * 4;
    c->serial = 0;
    c->dedup = DEDUP_AUTO;
    c->lambda_otf = 18.0f;
    c->lambda_full = 72.0f;
    c->hub_degree = 8192;
    cudaError_t e = cudaMallocHost((void**)&c->h_pinned, 64 * sizeof(int32_t));
    if (e != cudaSuccess) { delete c; return cuda_fail(e, "cudaMallocHost"); }

    cudaStream_t s = (cudaStream_t)stream;
    e = cudaMemsetAsync(c->d_hdr, 0, HDR_BYTES, s);
    if (e != cudaSuccess) { cudaFreeHost(c->h_pinned); delete c; return cuda_fail(e, "cudaMemsetAsync"); }
    if (split_cache) {
        // Row index of the dense part (tile sums live in the not yet used relabel table); the number
        // of dense nodes the caller sized the storage for must be the graph's.
        int32_t* d_cnt = c->d_hdr + HDR_WORDS;
        e = launch_build_row_index(GraphView{g->d_indptr, g->d_indices, g->num_nodes}, theta, c->d_row_index,
                                   (int32_t*)c->d_table, d_cnt, s);
        if (e == cudaSuccess) e = cudaMemcpyAsync(c->h_pinned, d_cnt, 2 * sizeof(int32_t), cudaMemcpyDeviceToHost, s);
        if (e == cudaSuccess) e = cudaStreamSynchronize(s);
        if (e != cudaSuccess) { cudaFreeHost(c->h_pinned); delete c; return cuda_fail(e, "row index"); }
        if ((int64_t)c->h_pinned[1] != dense_rows) {
            const long long got = c->h_pinned[1];
            cudaFreeHost(c->h_pinned);
            delete c;
            return fail(GS_ERR_ARG, "dense_rows = %lld, but %lld nodes have a degree above theta", (long long)dense_rows, got);
        }
    } else {
        e = launch_init_low_rows(GraphView{g->d_indptr, g->d_indices, g->num_nodes}, c->d_slots, c->pitch, c->W,
                                 c->num_caches, s);
        if (e != cudaSuccess) { cudaFreeHost(c->h_pinned); delete c; return cuda_fail(e, "pre-sample launch"); }
    }
    e = refresh_every_row(c, c->W, 0u, 1, s);
    if (e != cudaSuccess) { cudaFreeHost(c->h_pinned); delete c; return cuda_fail(e, "pre-sample launch"); }
    *out = c;
    return GS_OK;
}

gs_status gs_cache_init(const gs_graph* g, int32_t num_hops, const int32_t* fanouts, int32_t cache_width, uint64_t seed,
                        int32_t shared, void* d_cache_storage, size_t cache_bytes, void* stream, gs_cache** out) {
    return cache_init_impl(g, num_hops, fanouts, cache_width, seed, shared, -1, g ? g->num_nodes : 0, d_cache_storage,
                           cache_bytes, stream, out);
}

gs_status gs_cache_init_split(const gs_graph* g, int32_t num_hops, const int32_t* fanouts, int32_t cache_width,
                              uint64_t seed, int32_t shared, int32_t theta, int64_t dense_rows, void* d_cache_storage,
                              size_t cache_bytes, void* stream, gs_cache** out) {
    if (theta < 0) return fail(GS_ERR_ARG, "theta must be >= 0");
    return cache_init_impl(g, num_hops, fanouts, cache_width, seed, shared, theta, dense_rows, d_cache_storage,
                           cache_bytes, stream, out);
}

void gs_cache_destroy(gs_cache* c) {
    if (!c) return;
    if (c->h_pinned) cudaFreeHost(c->h_pinned);
    if (c->prof_events) {
        for (int i = 0; i < c->prof_cap * c->L * PROF_EVENTS_PER_STEP; ++i) cudaEventDestroy(c->prof_events[i]);
        delete[] c->prof_events;
    }
    delete c;
}

gs_status gs_cache_profile_begin(gs_cache* c, int32_t max_batches) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    if (max_batches < 1 || max_batches > 4096) return fail(GS_ERR_ARG, "max_batches outside [1, 4096]");
    if (c->prof_events) return fail(GS_ERR_ARG, "profiling is already on");
    const int n = max_batches * c->L * PROF_EVENTS_PER_STEP;
    c->prof_events = new (std::nothrow) cudaEvent_t[n];
    if (!c->prof_events) return fail(GS_ERR_ARG, "out of host memory");
    for (int i = 0; i < n; ++i) {
        cudaError_t e = cudaEventCreate(&c->prof_events[i]);
        if (e != cudaSuccess) {
            for (int j = 0; j < i; ++j) cudaEventDestroy(c->prof_events[j]);
            delete[] c->prof_events;
            c->prof_events = nullptr;
            return cuda_fail(e, "cudaEventCreate");
        }
    }
    c->prof_cap = max_batches;
    c->prof_used = 0;
    return GS_OK;
}

gs_status gs_cache_profile_end(gs_cache* c, void* stream, double* h_ms, int64_t* h_batches) {
    if (!c || !h_ms || !h_batches) return fail(GS_ERR_ARG, "NULL argument");
    if (!c->prof_events) return fail(GS_ERR_ARG, "profiling is not on");
    GS_CUDA(cudaStreamSynchronize((cudaStream_t)stream));
    for (int gI = 0; gI < PROF_GROUPS; ++gI) h_ms[gI] = 0.0;
    for (int b = 0; b < c->prof_used; ++b)
        for (int k = 0; k < c->L; ++k) {
            cudaEvent_t* ev = c->prof_events + ((size_t)b * c->L + k) * PROF_EVENTS_PER_STEP;
            for (int gI = 0; gI < PROF_GROUPS; ++gI) {
                float ms = 0.f;
                GS_CUDA(cudaEventElapsedTime(&ms, ev[gI], ev[gI + 1]));
                h_ms[gI] += ms;
            }
        }
    *h_batches = c->prof_used;
    for (int i = 0; i < c->prof_cap * c->L * PROF_EVENTS_PER_STEP; ++i) cudaEventDestroy(c->prof_events[i]);
    delete[] c->prof_events;
    c->prof_events = nullptr;
    c->prof_cap = c->prof_used = 0;
    return GS_OK;
}

gs_status gs_cache_set_dedup(gs_cache* c, int32_t method) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    if (method != DEDUP_DIRECT && method != DEDUP_HASH && method != DEDUP_SORT && method != DEDUP_AUTO) return fail(GS_ERR_ARG, "unknown dedup method %d", method);
    c->dedup = method;
    return GS_OK;
}

gs_status gs_cache_set_tuning(gs_cache* c, double lambda_otf, double lambda_full, int32_t hub_degree) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    if (lambda_otf > 0) c->lambda_otf = (float)lambda_otf;
    if (lambda_full > 0) c->lambda_full = (float)lambda_full;
    if (hub_degree > 0) c->hub_degree = hub_degree;
    return GS_OK;
}

// The stamp of a new batch: newer batches always win the atomicMin on the relabel table.
static uint32_t next_stamp(gs_cache* c, cudaStream_t s) {
    if (c->serial == 0xFFFFFFFEu) {  // stamp space used up: start over with a clean table
        if (cudaMemsetAsync(c->d_table, 0xFF, (size_t)c->graph->num_nodes * 8, s) != cudaSuccess) return 0;
        c->serial = 0;
    }
    c->serial += 1;
    return 0xFFFFFFFFu - c->serial;
}

// One hop of a node-sharded run, owner side: refresh + pick for a list of distinct nodes at one
// layer, the picks exported as rows of f ids.  Runs on the second header and leaves the relabel
// table alone, so it may come between the hops of this rank's own batch.
struct HopArgs {
    int32_t layer;
    int32_t* d_picks;   // [n][f], -1 padded
    const int32_t* d_n; // length of the list on the device (num_seeds is its bound then), or NULL
};

static gs_status sample_impl(gs_cache* c, const int32_t* d_seeds, int32_t num_seeds, gs_mode mode, double gamma,
                             uint32_t step, void* d_workspace, size_t workspace_bytes, cudaStream_t s,
                             gs_block* blocks, const int32_t** d_input_nodes, const int32_t** d_num_input_nodes,
                             const OutputBuffers* out = nullptr, const HopArgs* hop = nullptr) {
    const gs_graph* g = c->graph;
    const int L = hop ? 1 : c->L;
    int32_t* const hdr = hop ? c->d_hdr + HDR_OWNER : c->d_hdr;
    int32_t r;
    if (mode == GS_MODE_FCR || mode == GS_MODE_FBL) {
        r = c->W;
    } else if (mode == GS_MODE_OTF_FETCH) {
        r = 0;   // nothing is ever evicted; the per-layer fetch count is derived below
    } else {
        double rr = std::floor(gamma * (double)c->W + 0.5);
        r = rr < 0 ? 0 : (rr > c->W ? c->W : (int32_t)rr);
    }
    const Bounds b = make_bounds(g->num_nodes, L, hop ? c->fanouts + hop->layer : c->fanouts, num_seeds);
    const WorkspaceLayout w = make_layout(b, g->num_edges);
    if (workspace_bytes < w.total) return fail(GS_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, w.total);
    char* ws = (char*)d_workspace;
    int32_t* frontier = (int32_t*)(ws + w.frontier);
    int32_t* picked = (int32_t*)(ws + w.picked);
    int32_t* aux = (int32_t*)(ws + w.aux);
    int32_t* tiles_a = (int32_t*)(ws + w.tiles_a);
    int32_t* tiles_e = (int32_t*)(ws + w.tiles_e);
    if (out) {   // outputs go to the caller's buffers; only the scratch regions of `ws` are used
        if (!out->input_nodes || out->input_nodes_capacity < b.nb[L])
            return fail(GS_ERR_WORKSPACE, "input-node buffer holds %lld ids, %lld needed", (long long)out->input_nodes_capacity, (long long)b.nb[L]);
        for (int k = 0; k < L; ++k) {
            const int layer = L - 1 - k;
            if (!out->indptr[layer] || !out->indices[layer]) return fail(GS_ERR_ARG, "block buffers of layer %d are NULL", layer);
            if (out->indptr_capacity[layer] < b.nb[k] + 1 || out->indices_capacity[layer] < b.mb[k])
                return fail(GS_ERR_WORKSPACE, "block buffers of layer %d are too small: need %lld offsets and %lld indices",
                            layer, (long long)b.nb[k] + 1, (long long)b.mb[k]);
        }
        frontier = out->input_nodes;
    }

    uint32_t stamp = 0;
    if (!hop) {
        stamp = next_stamp(c, s);
        if (!stamp) return cuda_fail(cudaGetLastError(), "cudaMemsetAsync");
    }
    // the owner-side status word outlives the call: gs_shard_status reports (and clears) what any list
    // served since its last call has met
    if (hop) GS_CUDA(cudaMemsetAsync(hdr + HDR_STATUS + 1, 0, HDR_ONE - sizeof(int32_t), s));
    else GS_CUDA(cudaMemsetAsync(hdr, 0, HDR_ONE, s));

    const bool prof = !hop && c->prof_events && c->prof_used < c->prof_cap;
    for (int k = 0; k < L; ++k) {
        const int layer = hop ? hop->layer : L - 1 - k;
        // how this step finds first occurrences; key bounds grow with k, so AUTO never returns from the hash
        // table to the direct one inside a batch (the direct table is not maintained by the other methods)
        int32_t dedup = c->dedup;
        if (dedup == DEDUP_AUTO)
            dedup = (g->num_nodes * 8 > DEDUP_AUTO_TABLE_BYTES && b.nb[k] + b.mb[k] >= DEDUP_AUTO_MIN_KEYS) ? DEDUP_HASH : DEDUP_DIRECT;
        cudaEvent_t* ev = prof ? c->prof_events + ((size_t)c->prof_used * L + k) * PROF_EVENTS_PER_STEP : nullptr;
        if (ev) GS_CUDA(cudaEventRecord(ev[0], s));
        int32_t* blk_indptr = out ? out->indptr[layer] : (int32_t*)(ws + w.blk_indptr[k]);
        int32_t* blk_indices = out ? out->indices[layer] : (int32_t*)(ws + w.blk_indices[k]);

        CountParams C{};
        C.g = GraphView{g->d_indptr, g->d_indices, g->num_nodes};
        C.seeds = (k == 0) ? d_seeds : nullptr;
        C.frontier = frontier;
        C.hdr = hdr;
        C.k = k;
        C.f = c->fanouts[layer];
        C.n_host = num_seeds;
        C.d_n0 = hop ? hop->d_n : nullptr;
        C.blk_indptr = blk_indptr;
        C.tile_sums = tiles_a;
        C.table = c->d_table;
        C.stamp = stamp;
        C.no_stamp = hop ? 1 : 0;   // the seeds are stamped in the direct table with every dedup method: duplicates are caught before anything is refreshed
        // a partial refresh runs as scan + finish kernels; FCR (and r = 0) use the fused kernels
        int32_t n_fetch = 0;
        if (mode == GS_MODE_OTF_FETCH) {
            double nf = std::floor(gamma * (double)c->fanouts[layer] + 0.5);
            n_fetch = nf < 0 ? 0 : (nf > c->fanouts[layer] ? c->fanouts[layer] : (int32_t)nf);
        }
        // every batch runs as scan + finish kernels; a step that refreshes and fetches nothing (OTF
        // with r = 0, OTF Fetch with no fetch at this layer) has no scan items and skips the scan launch
        const bool fbl = (mode == GS_MODE_FBL);
        const bool scans = fbl || r > 0 || n_fetch > 0;
        C.W = fbl ? c->fanouts[layer] : (c->theta > c->W ? c->theta : c->W);   // rows above this degree are refreshed
        C.r = n_fetch > 0 ? n_fetch : (fbl ? c->fanouts[layer] : r);
        C.d_refresh_from = (c->shared && k > 0 && mode != GS_MODE_OTF_FETCH && !fbl) ? hdr + HDR_N + (k - 1) : nullptr;   // k = 0 for a single hop
        C.tile_sums2 = (int32_t*)(ws + w.tiles_a2);
        C.item_start = (int32_t*)(ws + w.item_start);
        C.items = (int4*)(ws + w.items);
        C.cand_count = (int32_t*)(ws + w.cand_count);
        C.scan_item_cap = w.scan_item_cap;
        GS_CUDA(launch_row_counts(C, b.nb[k], s));
        if (ev) GS_CUDA(cudaEventRecord(ev[1], s));

        StepParams P = step_params(c, layer, step);
        P.r = r;
        P.frontier = frontier;
        P.d_n = hdr + HDR_N + k;
        P.n_host = 0;
        P.d_refresh_from = (c->shared && k > 0) ? hdr + HDR_N + (k - 1) : nullptr;
        P.blk_indptr = blk_indptr;
        P.picked = picked;
        P.stamp = stamp;
        P.hub_entry = (int2*)(ws + w.hub_entry);
        P.hub_state = (int2*)(ws + w.hub_state);
        P.hub_items = (int32_t*)(ws + w.hub_items);
        P.hub_cand = (unsigned long long*)(ws + w.hub_cand);
        P.hub_counter = (unsigned long long*)(hdr + HDR_HUB64 + 2 * k);
        P.hub_cap = (int32_t)w.hub_cap;
        P.item_cap = (int32_t)w.item_cap;
        P.work_counter = hdr + HDR_WORK + k;
        P.work_counter2 = hdr + HDR_WORK2 + k;
        P.work_counter_scan = hdr + HDR_WORK3 + k;
        P.do_pick = 1;
        P.init_rows = 0;
        if (dedup != DEDUP_DIRECT) P.table = nullptr;   // positions are claimed after the step, from the picked array
        if (hop) {   // a shared cache refreshes every requested node: the same keys give the same row again
            P.table = nullptr;
            P.status = hdr + HDR_STATUS;
            P.stats = hdr + HDR_STAT_SLOW;
            P.d_refresh_from = nullptr;
        }
        if (n_fetch > 0) {           // scan + finish with FETCH keys; the finish kernel emits cache part + fetched part
            P.fetch = 1;
            P.r = n_fetch;
            P.word_fill = key_word(4, (uint32_t)layer);
            P.d_refresh_from = nullptr;
        }
        if (fbl) {   // W = r = f and FETCH keys; no cache row is touched
            P.fbl = 1;
            P.W = P.r = P.f;
            P.word_fill = key_word(4, (uint32_t)layer);
            P.d_refresh_from = nullptr;
        }
        if (P.r >= P.W) {
            // a full refill needs the whole top-W in the 64-entry candidate list: aim at the middle
            // of [W, 64] (for W = 32 about 1 % of the rows miss on either side and are rescanned)
            P.lambda_otf = c->lambda_full * (float)(P.W + SPLIT_CAND_CAP) / 144.0f;
        }
        P.item_start = C.item_start;
        P.items = C.items;
        P.d_items_total = hdr + HDR_ITEMS + k;
        P.cand_count = C.cand_count;
        P.cand = (unsigned long long*)(ws + w.cand);
        if (scans) {
            int64_t item_bound = b.nb[k] + g->num_edges / (4 * (int64_t)HUB_CHUNK_QUADS) + 1;
            GS_CUDA(launch_scan(P, item_bound, s));
        }
        if (ev) GS_CUDA(cudaEventRecord(ev[2], s));
        GS_CUDA(launch_finish(P, b.nb[k], s));
        if (ev) GS_CUDA(cudaEventRecord(ev[3], s));
        if (hop) {
            GS_CUDA(launch_export_picks(blk_indptr, picked, num_seeds, hdr + HDR_N, c->fanouts[layer], hop->d_picks, s));
            break;
        }

        RelabelParams R{};
        R.hdr = hdr;
        R.k = k;
        R.picked = picked;
        R.aux = aux;
        R.tile_sums = tiles_e;
        R.frontier = frontier;
        R.local = blk_indices;
        R.table = c->d_table;
        R.stamp = stamp;
        R.n_cap = b.nb[k + 1];
        R.method = dedup;
        R.scratch = (unsigned long long*)(ws + w.dedup);
        R.scratch_entries = w.dedup_entries;
        R.id_bits = 1;
        while (R.id_bits < 32 && ((int64_t)1 << R.id_bits) < g->num_nodes) R.id_bits += 1;
        GS_CUDA(launch_relabel(R, b.nb[k], b.mb[k], s));
        if (ev) GS_CUDA(cudaEventRecord(ev[4], s));

        gs_block& B = blocks[layer];
        B.max_dst = (int32_t)b.nb[k];
        B.max_src = (int32_t)b.nb[k + 1];
        B.max_edges = (int32_t)b.mb[k];
        B.d_num_dst = hdr + HDR_N + k;
        B.d_num_src = hdr + HDR_N + k + 1;
        B.d_num_edges = hdr + HDR_M + k;
        B.d_indptr = blk_indptr;
        B.d_indices = blk_indices;
    }
    if (prof) c->prof_used += 1;
    if (d_input_nodes) *d_input_nodes = frontier;
    if (d_num_input_nodes) *d_num_input_nodes = hdr + HDR_N + L;
    return GS_OK;
}

static gs_status check_batch_args(gs_cache* c, const int32_t* seeds, int32_t num_seeds, gs_mode mode, double gamma,
                                  uint32_t step, void* d_workspace, gs_block* blocks) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    if (!seeds) return fail(GS_ERR_ARG, "seeds is NULL");
    if (num_seeds < 1) return fail(GS_ERR_ARG, "num_seeds must be >= 1");
    if ((int64_t)num_seeds > c->graph->num_nodes) return fail(GS_ERR_ARG, "more seeds than nodes");
    if (mode != GS_MODE_FCR && mode != GS_MODE_OTF && mode != GS_MODE_FBL && mode != GS_MODE_OTF_FETCH)
        return fail(GS_ERR_ARG, "unknown mode %d", (int)mode);
    if ((mode == GS_MODE_OTF || mode == GS_MODE_OTF_FETCH) && !(gamma >= 0.0 && gamma <= 1.0))
        return fail(GS_ERR_ARG, "gamma outside [0, 1]");
    if (step == 0) return fail(GS_ERR_ARG, "step 0 is reserved for the pre-sample");
    if (!d_workspace) return fail(GS_ERR_ARG, "d_workspace is NULL");
    if (!aligned(d_workspace, 256)) return fail(GS_ERR_ALIGN, "d_workspace must be 256-byte aligned");
    if (!blocks) return fail(GS_ERR_ARG, "blocks is NULL");
    return GS_OK;
}

}  // extern "C"

namespace gs {
int32_t cache_num_hops(const gs_cache* c) { return c ? c->L : 0; }

gs_status cache_workspace_bytes(const gs_cache* c, int32_t num_seeds, size_t* bytes) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    return gs_workspace_bytes(c->graph, c->L, c->fanouts, num_seeds, bytes);
}

gs_status sample_batch_checked(gs_cache* c, const int32_t* d_seeds, int32_t num_seeds, gs_mode mode, double gamma,
                               uint32_t step, void* d_workspace, size_t workspace_bytes, cudaStream_t s,
                               gs_block* blocks, const int32_t** d_input_nodes, const int32_t** d_num_input_nodes,
                               const OutputBuffers* out) {
    gs_status st = check_batch_args(c, d_seeds, num_seeds, mode, gamma, step, d_workspace, blocks);
    if (st != GS_OK) return st;
    if (!aligned(d_seeds, 4)) return fail(GS_ERR_ALIGN, "d_seeds must be 4-byte aligned");
    return sample_impl(c, d_seeds, num_seeds, mode, gamma, step, d_workspace, workspace_bytes, s, blocks, d_input_nodes,
                       d_num_input_nodes, out);
}
}  // namespace gs

extern "C" {

gs_status gs_sample_batch(gs_cache* c, const int32_t* d_seeds, int32_t num_seeds, gs_mode mode, double gamma,
                          uint32_t step, void* d_workspace, size_t workspace_bytes, void* stream, gs_block* blocks,
                          const int32_t** d_input_nodes, const int32_t** d_num_input_nodes) {
    gs_status st = check_batch_args(c, d_seeds, num_seeds, mode, gamma, step, d_workspace, blocks);
    if (st != GS_OK) return st;
    if (!aligned(d_seeds, 4)) return fail(GS_ERR_ALIGN, "d_seeds must be 4-byte aligned");
    return sample_impl(c, d_seeds, num_seeds, mode, gamma, step, d_workspace, workspace_bytes, (cudaStream_t)stream,
                       blocks, d_input_nodes, d_num_input_nodes);
}

gs_status gs_cache_refresh_all(gs_cache* c, gs_mode mode, double gamma, uint32_t step, void* stream) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    if (mode != GS_MODE_FCR && mode != GS_MODE_OTF) return fail(GS_ERR_ARG, "only FCR and OTF refresh the cache");
    if (mode == GS_MODE_OTF && !(gamma >= 0.0 && gamma <= 1.0)) return fail(GS_ERR_ARG, "gamma outside [0, 1]");
    if (step == 0) return fail(GS_ERR_ARG, "step 0 is reserved for the pre-sample");
    int32_t r = c->W;
    if (mode == GS_MODE_OTF) {
        double rr = std::floor(gamma * (double)c->W + 0.5);
        r = rr < 0 ? 0 : (rr > c->W ? c->W : (int32_t)rr);
    }
    if (r == 0) return GS_OK;
    cudaStream_t s = (cudaStream_t)stream;
    GS_CUDA(cudaMemsetAsync(c->d_hdr, 0, HDR_ONE, s));
    GS_CUDA(refresh_every_row(c, r, step, 0, s));
    c->serial = 0;   // the table was reset: stamps start over
    return GS_OK;
}

/* ---------------------------------------------------------------- node-sharded sampling */

static gs_status shard_bucket_impl(const int32_t* d_nodes, int32_t n, const int32_t* d_n, int64_t num_nodes, int32_t world,
                                   int32_t capacity, int32_t* d_sorted, int32_t* d_slot, int32_t* d_counts, void* stream) {
    if (world < 1 || world > 64) return fail(GS_ERR_ARG, "world %d outside [1, 64]", world);
    if (num_nodes < 1 || num_nodes >= ((int64_t)1 << 31)) return fail(GS_ERR_ARG, "num_nodes outside [1, 2^31)");
    if (n < 0) return fail(GS_ERR_ARG, "n is negative");
    if (capacity < 0 || (int64_t)capacity * world >= ((int64_t)1 << 31)) return fail(GS_ERR_ARG, "capacity outside [0, 2^31 / world)");
    if (!d_counts || (n > 0 && (!d_nodes || !d_sorted || !d_slot))) return fail(GS_ERR_ARG, "NULL argument");
    const int32_t rows_per_shard = (int32_t)((num_nodes + world - 1) / world);
    GS_CUDA(launch_shard_bucket(d_nodes, n, d_n, rows_per_shard, world, capacity, d_sorted, d_slot, d_counts,
                                d_counts + 2 * world, (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_shard_bucket(const int32_t* d_nodes, int32_t n, int64_t num_nodes, int32_t world, int32_t* d_sorted,
                          int32_t* d_slot, int32_t* d_counts, void* stream) {
    return shard_bucket_impl(d_nodes, n, nullptr, num_nodes, world, 0, d_sorted, d_slot, d_counts, stream);
}

gs_status gs_shard_bucket_counted(const int32_t* d_nodes, const int32_t* d_n, int32_t n_bound, int64_t num_nodes,
                                  int32_t world, int32_t* d_sorted, int32_t* d_slot, int32_t* d_counts, void* stream) {
    if (!d_n) return fail(GS_ERR_ARG, "d_n is NULL");
    return shard_bucket_impl(d_nodes, n_bound, d_n, num_nodes, world, 0, d_sorted, d_slot, d_counts, stream);
}

gs_status gs_shard_bucket_fixed(const int32_t* d_nodes, const int32_t* d_n_or_null, int32_t n_bound, int64_t num_nodes,
                                int32_t world, int32_t capacity, int32_t* d_sorted, int32_t* d_slot, int32_t* d_counts,
                                void* stream) {
    if (capacity < 1) return fail(GS_ERR_ARG, "capacity must be >= 1");
    return shard_bucket_impl(d_nodes, n_bound, d_n_or_null, num_nodes, world, capacity, d_sorted, d_slot, d_counts, stream);
}

gs_status gs_shard_workspace_bytes(const gs_graph* g, int32_t fanout, int32_t max_nodes, size_t* bytes) {
    return gs_workspace_bytes(g, 1, &fanout, max_nodes, bytes);
}

static gs_status shard_sample_rows_impl(gs_cache* c, const int32_t* d_nodes, const int32_t* d_n, int32_t n, int32_t layer,
                                        gs_mode mode, double rate, uint32_t step, void* d_workspace, size_t workspace_bytes,
                                        void* stream, int32_t* d_picks) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    if (layer < 0 || layer >= c->L) return fail(GS_ERR_ARG, "layer %d outside [0, %d)", layer, c->L);
    if (n == 0) return GS_OK;
    if (!d_picks) return fail(GS_ERR_ARG, "d_picks is NULL");
    gs_block unused[GS_MAX_HOPS];
    gs_status st = check_batch_args(c, d_nodes, n, mode, rate, step, d_workspace, unused);
    if (st != GS_OK) return st;
    if (!aligned(d_nodes, 4) || !aligned(d_picks, 4)) return fail(GS_ERR_ALIGN, "node and pick arrays must be 4-byte aligned");
    HopArgs hop{layer, d_picks, d_n};
    return sample_impl(c, d_nodes, n, mode, rate, step, d_workspace, workspace_bytes, (cudaStream_t)stream, unused, nullptr,
                       nullptr, nullptr, &hop);
}

gs_status gs_shard_sample_rows(gs_cache* c, const int32_t* d_nodes, int32_t n, int32_t layer, gs_mode mode, double rate,
                               uint32_t step, void* d_workspace, size_t workspace_bytes, void* stream, int32_t* d_picks) {
    return shard_sample_rows_impl(c, d_nodes, nullptr, n, layer, mode, rate, step, d_workspace, workspace_bytes, stream, d_picks);
}

gs_status gs_shard_sample_rows_counted(gs_cache* c, const int32_t* d_nodes, const int32_t* d_n, int32_t n_bound, int32_t layer,
                                       gs_mode mode, double rate, uint32_t step, void* d_workspace, size_t workspace_bytes,
                                       void* stream, int32_t* d_picks) {
    if (!d_n) return fail(GS_ERR_ARG, "d_n is NULL");
    if (c && n_bound > 0 && (int64_t)n_bound > c->graph->num_nodes) n_bound = (int32_t)c->graph->num_nodes;   // a list of distinct nodes
    return shard_sample_rows_impl(c, d_nodes, d_n, n_bound, layer, mode, rate, step, d_workspace, workspace_bytes, stream, d_picks);
}

static gs_status check_merge_args(const int32_t* d_lists, const int32_t* d_counts, int32_t world, int32_t capacity,
                                  int64_t first_row, int64_t rows_owned, const int32_t* d_index, const int32_t* d_distinct) {
    if (world < 1 || world > 64) return fail(GS_ERR_ARG, "world %d outside [1, 64]", world);
    if (capacity < 1 || (int64_t)capacity * world >= ((int64_t)1 << 31)) return fail(GS_ERR_ARG, "capacity outside [1, 2^31 / world)");
    if (first_row < 0 || rows_owned < 1 || first_row + rows_owned > ((int64_t)1 << 31)) return fail(GS_ERR_ARG, "bad row range");
    if (!d_lists || !d_counts || !d_index || !d_distinct) return fail(GS_ERR_ARG, "NULL argument");
    return GS_OK;
}

gs_status gs_shard_merge(const int32_t* d_lists, const int32_t* d_counts, int32_t world, int32_t capacity, int64_t first_row,
                         int64_t rows_owned, int32_t* d_index, int32_t* d_distinct, int32_t* d_num_distinct, void* stream) {
    gs_status st = check_merge_args(d_lists, d_counts, world, capacity, first_row, rows_owned, d_index, d_distinct);
    if (st != GS_OK) return st;
    if (!d_num_distinct) return fail(GS_ERR_ARG, "d_num_distinct is NULL");
    GS_CUDA(launch_shard_merge(d_lists, d_counts, world, capacity, first_row, rows_owned, d_index, d_distinct, d_num_distinct,
                               (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_shard_fan_out(const int32_t* d_lists, const int32_t* d_counts, int32_t world, int32_t capacity, int64_t first_row,
                           int64_t rows_owned, int32_t* d_index, const int32_t* d_distinct, const int32_t* d_num_distinct,
                           const int32_t* d_rows, int32_t fanout, int32_t* d_out, void* stream) {
    gs_status st = check_merge_args(d_lists, d_counts, world, capacity, first_row, rows_owned, d_index, d_distinct);
    if (st != GS_OK) return st;
    if (!d_num_distinct || !d_rows || !d_out) return fail(GS_ERR_ARG, "NULL argument");
    if (fanout < 1 || fanout > GS_MAX_CACHE_WIDTH) return fail(GS_ERR_ARG, "fanout %d outside [1, %d]", fanout, GS_MAX_CACHE_WIDTH);
    int64_t bound = (int64_t)world * capacity;
    if (bound > rows_owned) bound = rows_owned;
    GS_CUDA(launch_shard_fan_out(d_lists, d_counts, world, capacity, first_row, rows_owned, d_index, d_distinct, (int32_t)bound,
                                 d_rows, d_num_distinct, fanout, d_out, (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_shard_status(gs_cache* c, void* stream) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    cudaStream_t s = (cudaStream_t)stream;
    GS_CUDA(cudaMemcpyAsync(c->h_pinned, c->d_hdr + HDR_OWNER + HDR_STATUS, sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    GS_CUDA(cudaStreamSynchronize(s));
    const int status = c->h_pinned[0];
    if (status != 0) GS_CUDA(cudaMemsetAsync(c->d_hdr + HDR_OWNER + HDR_STATUS, 0, sizeof(int32_t), s));
    if (status == GS_ERR_RANGE) return fail(GS_ERR_RANGE, "a requested node id is outside [0, num_nodes)");
    if (status != 0) return fail(GS_ERR_CUDA, "unexpected device status %d", status);
    return GS_OK;
}

static gs_status shard_extend_impl(gs_cache* c, int32_t k, const int32_t* d_seeds, int32_t num_seeds, const int32_t* d_reply,
                                   int32_t reply_rows, const int32_t* d_slot, void* d_workspace, size_t workspace_bytes,
                                   void* stream, gs_block* block, const int32_t** d_frontier) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    if (k < 0 || k >= c->L) return fail(GS_ERR_ARG, "hop %d outside [0, %d)", k, c->L);
    if (!d_reply || !block) return fail(GS_ERR_ARG, "NULL argument");
    if (!d_workspace || !aligned(d_workspace, 256)) return fail(GS_ERR_ALIGN, "d_workspace must be 256-byte aligned");
    const gs_graph* g = c->graph;
    cudaStream_t s = (cudaStream_t)stream;
    if (k == 0) {
        if (!d_seeds) return fail(GS_ERR_ARG, "seeds is NULL");
        if (num_seeds < 1 || (int64_t)num_seeds > g->num_nodes) return fail(GS_ERR_ARG, "num_seeds outside [1, num_nodes]");
        const uint32_t stamp = next_stamp(c, s);
        if (!stamp) return cuda_fail(cudaGetLastError(), "cudaMemsetAsync");
        c->shard_stamp = stamp;
        c->shard_seeds = num_seeds;
        GS_CUDA(cudaMemsetAsync(c->d_hdr, 0, HDR_ONE, s));
    } else if (c->shard_seeds < 1) {
        return fail(GS_ERR_ARG, "hop %d before hop 0", k);
    }
    const int L = c->L, layer = L - 1 - k;
    const Bounds b = make_bounds(g->num_nodes, L, c->fanouts, c->shard_seeds);
    const WorkspaceLayout w = make_layout(b, g->num_edges);
    if (workspace_bytes < w.total) return fail(GS_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, w.total);
    char* ws = (char*)d_workspace;
    int32_t* frontier = (int32_t*)(ws + w.frontier);
    int32_t* picked = (int32_t*)(ws + w.picked);
    int32_t* blk_indptr = (int32_t*)(ws + w.blk_indptr[k]);
    int32_t* blk_indices = (int32_t*)(ws + w.blk_indices[k]);

    CountParams C{};
    C.g = GraphView{g->d_indptr, g->d_indices, g->num_nodes};
    C.seeds = (k == 0) ? d_seeds : nullptr;
    C.frontier = frontier;
    C.hdr = c->d_hdr;
    C.k = k;
    C.f = c->fanouts[layer];
    C.n_host = c->shard_seeds;
    C.blk_indptr = blk_indptr;
    C.tile_sums = (int32_t*)(ws + w.tiles_a);
    C.table = c->d_table;
    C.stamp = c->shard_stamp;
    C.W = c->W;
    C.r = 0;
    C.tile_sums2 = (int32_t*)(ws + w.tiles_a2);
    C.item_start = (int32_t*)(ws + w.item_start);
    C.items = (int4*)(ws + w.items);
    C.cand_count = (int32_t*)(ws + w.cand_count);
    C.scan_item_cap = w.scan_item_cap;
    C.reply = d_reply;
    C.reply_rows = reply_rows;
    C.slot = d_slot;
    GS_CUDA(launch_row_counts(C, b.nb[k], s));
    // first occurrences are found as in gs_sample_batch: the direct table takes its claims while the picks are
    // imported, the other methods work from the picked array afterwards
    int32_t dedup = c->dedup;
    if (dedup == DEDUP_AUTO)
        dedup = (g->num_nodes * 8 > DEDUP_AUTO_TABLE_BYTES && b.nb[k] + b.mb[k] >= DEDUP_AUTO_MIN_KEYS) ? DEDUP_HASH : DEDUP_DIRECT;
    GS_CUDA(launch_import_picks(c->d_hdr, k, (int32_t)b.nb[k], C.f, d_reply, reply_rows, d_slot, blk_indptr, picked,
                                dedup == DEDUP_DIRECT ? c->d_table : nullptr, c->shard_stamp, g->num_nodes,
                                c->d_hdr + HDR_STATUS, s));
    RelabelParams R{};
    R.hdr = c->d_hdr;
    R.k = k;
    R.picked = picked;
    R.aux = (int32_t*)(ws + w.aux);
    R.tile_sums = (int32_t*)(ws + w.tiles_e);
    R.frontier = frontier;
    R.local = blk_indices;
    R.table = c->d_table;
    R.stamp = c->shard_stamp;
    R.n_cap = b.nb[k + 1];
    R.method = dedup;
    R.scratch = (unsigned long long*)(ws + w.dedup);
    R.scratch_entries = w.dedup_entries;
    R.id_bits = 1;
    while (R.id_bits < 32 && ((int64_t)1 << R.id_bits) < g->num_nodes) R.id_bits += 1;
    GS_CUDA(launch_relabel(R, b.nb[k], b.mb[k], s));

    gs_block& B = *block;
    B.max_dst = (int32_t)b.nb[k];
    B.max_src = (int32_t)b.nb[k + 1];
    B.max_edges = (int32_t)b.mb[k];
    B.d_num_dst = c->d_hdr + HDR_N + k;
    B.d_num_src = c->d_hdr + HDR_N + k + 1;
    B.d_num_edges = c->d_hdr + HDR_M + k;
    B.d_indptr = blk_indptr;
    B.d_indices = blk_indices;
    if (d_frontier) *d_frontier = frontier;
    return GS_OK;
}

gs_status gs_shard_extend(gs_cache* c, int32_t k, const int32_t* d_seeds, int32_t num_seeds, const int32_t* d_reply,
                          const int32_t* d_slot, void* d_workspace, size_t workspace_bytes, void* stream, gs_block* block,
                          const int32_t** d_frontier) {
    return shard_extend_impl(c, k, d_seeds, num_seeds, d_reply, 0, d_slot, d_workspace, workspace_bytes, stream, block, d_frontier);
}

gs_status gs_shard_extend_fixed(gs_cache* c, int32_t k, const int32_t* d_seeds, int32_t num_seeds, const int32_t* d_reply,
                                int32_t reply_rows, const int32_t* d_slot, void* d_workspace, size_t workspace_bytes,
                                void* stream, gs_block* block, const int32_t** d_frontier) {
    if (reply_rows < 1) return fail(GS_ERR_ARG, "reply_rows must be >= 1");
    if (!d_slot) return fail(GS_ERR_ARG, "d_slot is NULL");
    return shard_extend_impl(c, k, d_seeds, num_seeds, d_reply, reply_rows, d_slot, d_workspace, workspace_bytes, stream, block,
                             d_frontier);
}

gs_status gs_gather_rows(const void* d_src, gs_dtype dtype, int32_t row_elems, int64_t src_ld, int64_t first_row,
                         int64_t src_rows, const int32_t* d_ids, const int32_t* d_count_or_null, int32_t count_bound, void* d_out,
                         int64_t out_ld, void* stream) {
    if (dtype != GS_F32 && dtype != GS_BF16) return fail(GS_ERR_ARG, "unknown dtype %d", (int)dtype);
    const int64_t eb = dtype == GS_BF16 ? 2 : 4;
    if (count_bound < 0) return fail(GS_ERR_ARG, "count_bound is negative");
    if (count_bound == 0) return GS_OK;
    if (!d_src || !d_ids || !d_out) return fail(GS_ERR_ARG, "NULL argument");
    if (row_elems < 1 || src_ld < row_elems || out_ld < row_elems) return fail(GS_ERR_ARG, "bad row size or pitch");
    if (first_row < 0 || src_rows < 1) return fail(GS_ERR_ARG, "first_row is negative or the source has no rows");
    if (!aligned(d_src, (size_t)eb) || !aligned(d_out, (size_t)eb) || !aligned(d_ids, 4)) return fail(GS_ERR_ALIGN, "misaligned argument");
    // ids are global; the source holds rows first_row, first_row + 1, ...: address row 0 where it would be
    const uintptr_t base = (uintptr_t)d_src - (uintptr_t)(first_row * src_ld * eb);
    GS_CUDA(launch_gather((const void*)base, src_ld * eb, (int64_t)row_elems * eb, d_ids, d_count_or_null, count_bound, d_out,
                          out_ld * eb, 0, first_row, first_row + src_rows, (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_gather_rows_peer(const void* const* h_shard_bases, int32_t world, int64_t num_rows, gs_dtype dtype,
                              int32_t row_elems, int64_t src_ld, const int32_t* d_ids, const int32_t* d_count_or_null,
                              int32_t count_bound, void* d_out, int64_t out_ld, void* stream) {
    if (dtype != GS_F32 && dtype != GS_BF16) return fail(GS_ERR_ARG, "unknown dtype %d", (int)dtype);
    const int64_t eb = dtype == GS_BF16 ? 2 : 4;
    if (world < 1 || world > 64) return fail(GS_ERR_ARG, "world %d outside [1, 64]", world);
    if (num_rows < 1 || num_rows >= ((int64_t)1 << 31)) return fail(GS_ERR_ARG, "num_rows outside [1, 2^31)");
    if (count_bound < 0) return fail(GS_ERR_ARG, "count_bound is negative");
    if (count_bound == 0) return GS_OK;
    if (!h_shard_bases || !d_ids || !d_out) return fail(GS_ERR_ARG, "NULL argument");
    if (row_elems < 1 || src_ld < row_elems || out_ld < row_elems) return fail(GS_ERR_ARG, "bad row size or pitch");
    const int64_t rows_per_shard = (num_rows + world - 1) / world;
    for (int o = 0; o < world; ++o) {
        const bool empty = (int64_t)o * rows_per_shard >= num_rows;   // a trailing shard may own no row
        if (!h_shard_bases[o] && !empty) return fail(GS_ERR_ARG, "shard %d has no base address", o);
        if (!aligned(h_shard_bases[o], (size_t)eb)) return fail(GS_ERR_ALIGN, "shard %d is misaligned", o);
    }
    if (!aligned(d_out, (size_t)eb) || !aligned(d_ids, 4)) return fail(GS_ERR_ALIGN, "misaligned argument");
    GS_CUDA(launch_gather_sharded(h_shard_bases, world, num_rows, rows_per_shard, src_ld * eb, (int64_t)row_elems * eb, d_ids,
                                  d_count_or_null, count_bound, d_out, out_ld * eb, (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_batch_counts(gs_cache* c, void* stream, int32_t* h_num_nodes, int32_t* h_num_edges) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    cudaStream_t s = (cudaStream_t)stream;
    GS_CUDA(cudaMemcpyAsync(c->h_pinned, c->d_hdr, (size_t)(HDR_M + GS_MAX_HOPS) * 4, cudaMemcpyDeviceToHost, s));
    GS_CUDA(cudaStreamSynchronize(s));
    const int status = c->h_pinned[HDR_STATUS];
    if (h_num_nodes)
        for (int k = 0; k <= c->L; ++k) h_num_nodes[k] = c->h_pinned[HDR_N + k];
    if (h_num_edges)
        for (int l = 0; l < c->L; ++l) h_num_edges[l] = c->h_pinned[HDR_M + (c->L - 1 - l)];
    if (status == GS_ERR_RANGE) return fail(GS_ERR_RANGE, "a seed id is outside [0, num_nodes)");
    if (status == GS_ERR_DUP_SEED) return fail(GS_ERR_DUP_SEED, "duplicate seed id in the batch");
    if (status != 0) return fail(GS_ERR_CUDA, "unexpected device status %d", status);
    return GS_OK;
}

gs_status gs_batch_stats(gs_cache* c, void* stream, int64_t* h_stats) {
    if (!c || !h_stats) return fail(GS_ERR_ARG, "NULL argument");
    cudaStream_t s = (cudaStream_t)stream;
    GS_CUDA(cudaMemcpyAsync(c->h_pinned, c->d_hdr + HDR_STAT_SLOW, 4 * sizeof(int32_t), cudaMemcpyDeviceToHost, s));
    GS_CUDA(cudaStreamSynchronize(s));
    for (int i = 0; i < 4; ++i) h_stats[i] = (int64_t)(uint32_t)c->h_pinned[i];
    return GS_OK;
}

gs_status gs_sync_status(gs_cache* c, void* stream) { return gs_batch_counts(c, stream, nullptr, nullptr); }

gs_status gs_sample_batch_host(gs_cache* c, const int32_t* h_seeds, int32_t num_seeds, gs_mode mode, double gamma,
                               uint32_t step, void* d_workspace, size_t workspace_bytes, void* stream, gs_block* blocks,
                               const int32_t** d_input_nodes, int32_t* h_num_nodes, int32_t* h_num_edges) {
    gs_status st = check_batch_args(c, h_seeds, num_seeds, mode, gamma, step, d_workspace, blocks);
    if (st != GS_OK) return st;
    // The seeds are staged in the relabel scratch array: its first writer (step 0's
    // first-occurrence kernel) runs after the row-count kernel has copied the seeds out.
    const Bounds b = make_bounds(c->graph->num_nodes, c->L, c->fanouts, num_seeds);
    const WorkspaceLayout w = make_layout(b, c->graph->num_edges);
    if (workspace_bytes < w.total) return fail(GS_ERR_WORKSPACE, "workspace has %zu bytes, %zu needed", workspace_bytes, w.total);
    int32_t* d_stage = (int32_t*)((char*)d_workspace + w.aux);
    cudaStream_t s = (cudaStream_t)stream;
    GS_CUDA(cudaMemcpyAsync(d_stage, h_seeds, (size_t)num_seeds * 4, cudaMemcpyHostToDevice, s));
    st = sample_impl(c, d_stage, num_seeds, mode, gamma, step, d_workspace, workspace_bytes, s, blocks, d_input_nodes, nullptr);
    if (st != GS_OK) return st;
    return gs_batch_counts(c, stream, h_num_nodes, h_num_edges);
}

gs_status gs_gather_features(const gs_graph* g, const int32_t* d_ids, const int32_t* d_count_or_null, int32_t count_bound,
                             void* d_out, int64_t out_ld, void* stream) {
    if (!g) return fail(GS_ERR_ARG, "graph is NULL");
    if (!g->d_features) return fail(GS_ERR_ARG, "the graph was created without features");
    if (count_bound < 0) return fail(GS_ERR_ARG, "count_bound is negative");
    if (count_bound == 0) return GS_OK;  // nothing to copy; an empty output may have no address
    if (!d_ids || !d_out) return fail(GS_ERR_ARG, "d_ids or d_out is NULL");
    if (out_ld < g->feat_dim) return fail(GS_ERR_ARG, "out_ld %lld < feat_dim %d", (long long)out_ld, g->feat_dim);
    if (!aligned(d_out, (size_t)g->elem_bytes)) return fail(GS_ERR_ALIGN, "d_out must be aligned to the element size");
    if (!aligned(d_ids, 4)) return fail(GS_ERR_ALIGN, "d_ids must be 4-byte aligned");
    GS_CUDA(launch_gather(g->d_features, g->feat_ld * g->elem_bytes, (int64_t)g->feat_dim * g->elem_bytes, d_ids,
                          d_count_or_null, count_bound, d_out, out_ld * g->elem_bytes, g->gather_blocks_per_sm, 0,
                          g->num_nodes, (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_cache_read_rows(const gs_cache* c, int32_t layer, const int32_t* d_nodes, int32_t n, int32_t* d_out, void* stream) {
    if (!c) return fail(GS_ERR_ARG, "cache is NULL");
    if (layer < 0 || layer >= c->L) return fail(GS_ERR_ARG, "layer %d outside [0, %d)", layer, c->L);
    if (n < 0 || (n > 0 && (!d_nodes || !d_out))) return fail(GS_ERR_ARG, "bad node list");
    const int32_t ci = c->shared ? 0 : layer;
    const int32_t* slots = c->d_slots + (size_t)ci * (size_t)c->rows * c->pitch;
    GS_CUDA(launch_read_rows(slots, c->d_row_index, c->pitch, c->W, d_nodes, n, d_out, (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_cache_export_bytes(const gs_cache* c, size_t* bytes) {
    if (!c || !bytes) return fail(GS_ERR_ARG, "NULL argument");
    *bytes = c->slot_bytes;
    return GS_OK;
}

gs_status gs_cache_export(const gs_cache* c, void* d_dst, size_t bytes, void* stream) {
    if (!c || !d_dst) return fail(GS_ERR_ARG, "NULL argument");
    if (bytes < c->slot_bytes) return fail(GS_ERR_WORKSPACE, "export buffer has %zu bytes, %zu needed", bytes, c->slot_bytes);
    GS_CUDA(cudaMemcpyAsync(d_dst, c->d_slots, c->slot_bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return GS_OK;
}

gs_status gs_cache_import(gs_cache* c, const void* d_src, size_t bytes, void* stream) {
    if (!c || !d_src) return fail(GS_ERR_ARG, "NULL argument");
    if (bytes != c->slot_bytes) return fail(GS_ERR_WORKSPACE, "import blob has %zu bytes, %zu expected", bytes, c->slot_bytes);
    GS_CUDA(cudaMemcpyAsync(c->d_slots, d_src, c->slot_bytes, cudaMemcpyDeviceToDevice, (cudaStream_t)stream));
    return GS_OK;
}

}  // extern "C"
