// Host-side descriptors shared by the C ABI and the kernel launchers.
#pragma once
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "../../include/gs.h"

namespace gs {

// ---- device state header at the start of the cache storage (int32 words) ----
constexpr int HDR_STATUS = 0;
constexpr int HDR_N = 1;                         // n_0 .. n_L              (GS_MAX_HOPS + 1 words)
constexpr int HDR_M = HDR_N + GS_MAX_HOPS + 1;   // m_k by sampling step    (GS_MAX_HOPS words)
constexpr int HDR_WORK = HDR_M + GS_MAX_HOPS;    // work-stealing counters  (GS_MAX_HOPS words)
constexpr int HDR_HUBS = HDR_WORK + GS_MAX_HOPS; // hub list lengths
constexpr int HDR_TICKET_A = HDR_HUBS + GS_MAX_HOPS;
constexpr int HDR_TICKET_E = HDR_TICKET_A + GS_MAX_HOPS;
constexpr int HDR_WORK2 = HDR_TICKET_E + GS_MAX_HOPS;  // work counters of the hub-chunk kernel
constexpr int HDR_ITEMS = HDR_WORK2 + GS_MAX_HOPS;     // scan work items per step (split OTF path)
constexpr int HDR_WORK3 = HDR_ITEMS + GS_MAX_HOPS;     // work counters of the scan kernel
constexpr int HDR_STAT_SLOW = HDR_WORK3 + GS_MAX_HOPS;    // nodes whose refill was retried by one warp (whole batch)
constexpr int HDR_STAT_QUEUED = HDR_STAT_SLOW + 1;        // nodes handed to the chunked hub kernel
constexpr int HDR_STAT_REFRESHED = HDR_STAT_QUEUED + 1;   // nodes refreshed
constexpr int HDR_STAT_QUADS = HDR_STAT_REFRESHED + 1;    // Philox blocks the scan kernel has to evaluate
constexpr int HDR_WORDS = HDR_STAT_QUADS + 1;
constexpr int HDR_HUB64 = 128;                   // 64-bit (hubs << 32 | chunks) counters, one per launch
constexpr size_t HDR_ONE = 1024;                 // bytes of one header
constexpr int HDR_OWNER = (int)(HDR_ONE / 4);    // word offset of the second header: owner-side hops of a sharded run
constexpr size_t HDR_BYTES = 2 * HDR_ONE;        // both headers, at the start of the cache storage
static_assert(HDR_WORDS <= HDR_HUB64, "header words overlap the 64-bit counters");
static_assert((HDR_HUB64 + 2 * GS_MAX_HOPS) * 4 <= HDR_ONE, "header too small");

#ifndef GS_SCAN_CHUNK_QUADS
#define GS_SCAN_CHUNK_QUADS 1024
#endif
constexpr int HUB_CHUNK_QUADS = GS_SCAN_CHUNK_QUADS;   // one scan work item = 4 x this many edge offsets
constexpr int HUB_MIN_DEGREE = 4096;    // lowest degree at which a node may be split over warps
constexpr int HUB_CAND_CAP = 128;       // candidate entries per hub (same as a warp's buffer)

constexpr int SPLIT_CAND_CAP = 64;      // candidates kept per node by the split OTF path (two per lane)
constexpr int SMALL_DEGREE = 128;       // up to here a refresh needs no threshold scan: one Philox per lane covers the row

constexpr int SCAN_A_TILE = 1024;  // frontier nodes per tile of the row-count scan
constexpr int SCAN_E_TILE = 4096;  // picked edges per tile of the first-occurrence scan

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

// Entries of the batch-sized hash table for n + m keys (load factor at most 2/3).
__host__ __device__ inline int64_t dedup_hash_capacity(int64_t keys) {
    return (keys + keys / 2 + 64) & ~(int64_t)1;
}
// 8-byte scratch entries the sort needs for `keys` pairs: two key buffers, the digit counters of every
// 4096-key tile, one run-head word per 1024 keys, a ticket and the 256 digit totals.
__host__ __device__ inline int64_t dedup_sort_entries(int64_t keys) {
    const int64_t tiles = (keys + 4095) / 4096 + 1, tiles1k = (keys + 1023) / 1024 + 1;
    return 2 * keys + 64 + (256 * tiles + tiles1k + 1024) / 2 + 8;
}

struct Bounds {
    int32_t L;
    int64_t nb[GS_MAX_HOPS + 1];  // upper bound of n_k
    int64_t mb[GS_MAX_HOPS];      // upper bound of m_k (by sampling step)
};

inline Bounds make_bounds(int64_t N, int32_t L, const int32_t* fanouts, int64_t seeds) {
    Bounds b{};
    b.L = L;
    b.nb[0] = seeds < N ? seeds : N;
    for (int k = 0; k < L; ++k) {
        b.mb[k] = b.nb[k] * fanouts[L - 1 - k];
        int64_t nn = b.nb[k] + b.mb[k];
        b.nb[k + 1] = nn < N ? nn : N;
    }
    return b;
}

struct WorkspaceLayout {
    size_t frontier;
    size_t blk_indptr[GS_MAX_HOPS];   // by sampling step
    size_t blk_indices[GS_MAX_HOPS];  // by sampling step
    size_t picked, aux, tiles_a, tiles_e;
    size_t hub_entry, hub_state, hub_items, hub_cand;
    int64_t hub_cap, item_cap;
    size_t tiles_a2, item_start, items, cand_count, cand;   // split OTF path
    size_t dedup;
    int64_t dedup_entries;
    int64_t scan_item_cap;
    size_t total;
};

// Hubs are nodes with degree > HUB_MIN_DEGREE or more; their number among distinct frontier
// nodes is bounded by num_edges / HUB_MIN_DEGREE, their chunks by num_edges / chunk + hubs.
inline void hub_caps(int64_t num_edges, int64_t max_n, int64_t* hub_cap, int64_t* item_cap) {
    int64_t h = num_edges / HUB_MIN_DEGREE + 1;
    if (h > max_n) h = max_n;
    *hub_cap = h;
    *item_cap = num_edges / (4 * (int64_t)HUB_CHUNK_QUADS) + h + 1;
}

inline WorkspaceLayout make_layout(const Bounds& b, int64_t num_edges) {
    WorkspaceLayout w{};
    size_t off = 0;
    auto take = [&](size_t bytes) { size_t o = off; off = align_up(off + bytes, 256); return o; };
    w.frontier = take((size_t)b.nb[b.L] * 4);
    int64_t max_m = 0, max_n = 0;
    for (int k = 0; k < b.L; ++k) {
        w.blk_indptr[k] = take(((size_t)b.nb[k] + 1) * 4);
        w.blk_indices[k] = take((size_t)b.mb[k] * 4 + 16);
        if (b.mb[k] > max_m) max_m = b.mb[k];
        if (b.nb[k] > max_n) max_n = b.nb[k];
    }
    w.picked = take((size_t)max_m * 4 + 16);
    w.aux = take((size_t)max_m * 4 + 16);
    w.tiles_a = take(((size_t)max_n / SCAN_A_TILE + 2) * 4);
    w.tiles_e = take(((size_t)max_m / SCAN_E_TILE + 2) * 4);
    hub_caps(num_edges, max_n, &w.hub_cap, &w.item_cap);
    w.hub_entry = take((size_t)w.hub_cap * 8);
    w.hub_state = take((size_t)w.hub_cap * 8);
    w.hub_items = take((size_t)w.item_cap * 4);
    w.hub_cand = take((size_t)w.hub_cap * HUB_CAND_CAP * 8);
    w.tiles_a2 = take(((size_t)max_n / SCAN_A_TILE + 2) * 4);
    w.item_start = take(((size_t)max_n + 1) * 4);
    w.scan_item_cap = max_n + num_edges / (4 * (int64_t)HUB_CHUNK_QUADS) + 1;
    w.items = take((size_t)w.scan_item_cap * sizeof(int4));
    w.cand_count = take((size_t)max_n * 4);
    w.cand = take((size_t)max_n * SPLIT_CAND_CAP * 8);
    w.dedup = w.cand;   // free once the step's picks are written: scratch of the alternative dedup methods
    {
        int64_t need = 0;
        for (int k = 0; k < b.L; ++k) {
            const int64_t keys = b.nb[k] + b.mb[k];
            const int64_t e = dedup_sort_entries(keys) > dedup_hash_capacity(keys) ? dedup_sort_entries(keys) : dedup_hash_capacity(keys);
            if (e > need) need = e;
        }
        w.dedup_entries = need;
        const size_t have = off - w.cand;
        if ((size_t)need * 8 > have) off = align_up(w.cand + (size_t)need * 8, 256);
    }
    w.total = off;
    return w;
}

// ---- kernel parameter blocks ----
struct GraphView {
    const int64_t* indptr;
    const int32_t* indices;
    int64_t num_nodes;
};

struct StepParams {
    GraphView g;
    int32_t* slots;        // this step's cache: [rows][pitch]; row of node v = v, or row_index[v] in a split cache
    const int32_t* row_index;  // split cache only: cache row of each node, -1 for the sparse part (degree <= theta)
    int32_t theta;         // split cache: nodes with degree <= theta are sampled from the graph; -1 = no split
    uint32_t word_fetch;   // (FETCH << 8) | layer, the key word of the sparse part
    int32_t pitch, W, f, r;
    uint32_t step, key0, key1;
    uint32_t rk[20];       // Philox round keys derived from (key0, key1)
    uint32_t word_fill, word_evict, word_pick;  // (purpose << 8) | tag
    const int32_t* frontier;     // NULL: identity (node id = position)
    const int32_t* d_n;          // device count of frontier nodes, or NULL -> n_host
    int32_t n_host;
    const int32_t* d_refresh_from;  // device scalar: positions below it are not refreshed; NULL -> 0
    const int32_t* blk_indptr;   // final offsets of each node's picks
    int32_t* picked;             // global ids of the picks
    unsigned long long* table;   // relabel table, (stamp << 32) | position; NULL: picks are not registered (owner side of a sharded run)
    uint32_t stamp;
    // hubs: nodes whose scan is split into chunks over many warps
    int2* hub_entry;                 // (frontier position, first chunk)
    int2* hub_state;                 // (candidates appended, chunks finished)
    int32_t* hub_items;              // chunk -> hub entry
    unsigned long long* hub_cand;    // [hub][HUB_CAND_CAP] (key << 32 | offset)
    unsigned long long* hub_counter; // (entries << 32) | chunks
    int32_t hub_cap, item_cap;
    int32_t* work_counter;
    int32_t* work_counter2;
    int32_t* work_counter_scan;
    // split OTF path: scan work items (one per 4096-offset chunk of a refreshed node) and the
    // per-node candidate lists they produce
    const int32_t* item_start;       // [n+1] first item of each frontier position
    const int4* items;               // item -> (frontier position, node, degree, chunk of the node's row)
    const int32_t* d_items_total;
    int32_t* cand_count;             // [n]
    unsigned long long* cand;        // [n][SPLIT_CAND_CAP]
    int32_t* status;
    int32_t* stats;                  // header words HDR_STAT_*: rare-event counters
    int32_t do_pick, init_rows;
    int32_t fetch;                   // OTF Fetch: r neighbours come from the graph, f - r from the cache; no row is written
    int32_t fbl;                     // Full Batch Load: W = r = f, no cache row is read or written
    float lambda_otf, lambda_full;
    int32_t hub_degree;
};

struct CountParams {
    GraphView g;
    const int32_t* seeds;    // step 0: copied into frontier; else NULL
    int32_t* frontier;
    int32_t* hdr;            // device header words
    int32_t k;               // sampling step
    int32_t f;
    int32_t n_host;          // step 0 only
    int32_t* blk_indptr;
    int32_t* tile_sums;
    unsigned long long* table;
    uint32_t stamp;
    // also lays out the scan work items of the refreshed nodes (rows above SMALL_DEGREE, r > 0)
    int32_t W, r;
    const int32_t* d_refresh_from;
    int32_t* tile_sums2;
    int32_t* item_start;
    int4* items;
    int32_t* cand_count;
    int64_t scan_item_cap;
    // sharded sampling
    int32_t no_stamp;        // owner side: step 0 neither checks duplicates nor touches the relabel table
    const int32_t* reply;    // requester side: picks by row [rows][f], -1 padded; row lengths come from here, not from degrees
    const int32_t* slot;     // requester side: row of `reply` that belongs to frontier position p
    int32_t reply_rows;      // rows `reply` holds when its segments have a fixed pitch; 0: exactly n_k rows
    const int32_t* d_n0;     // step 0: the list's length on the device (n_host is its bound then), or NULL
};

// How the position of an id's first occurrence in "frontier ++ picked" is found (S3).
enum DedupMethod : int32_t {
    DEDUP_DIRECT = 0,   // direct-address table uint64[num_nodes]; the pick kernels claim positions with atomicMin
    DEDUP_HASH = 1,     // open-addressing hash table sized to the batch (1.5 x (n_k + m_k) entries), rebuilt per step
    DEDUP_SORT = 2,     // stable radix sort of (id, position) pairs; the head of each run of equal ids is the first occurrence
    DEDUP_AUTO = 3      // per sampling step: the hash table where the direct table is far larger than L2 and the step is large
};
// DEDUP_AUTO takes the hash table for a step when the direct table (8 bytes per node) exceeds this many bytes
// - it no longer stays in the 126 MB L2 - and the step may hold at least this many keys (frontier + picks bound);
// measured on B200: below either limit the direct table wins.
constexpr int64_t DEDUP_AUTO_TABLE_BYTES = (int64_t)64 << 20;
constexpr int64_t DEDUP_AUTO_MIN_KEYS = (int64_t)1 << 19;

struct RelabelParams {
    int32_t* hdr;
    int32_t k;
    const int32_t* picked;
    int32_t* aux;
    int32_t* tile_sums;
    int32_t* frontier;
    int32_t* local;
    unsigned long long* table;       // DEDUP_DIRECT only
    uint32_t stamp;
    int64_t n_cap;
    int32_t method;
    unsigned long long* scratch;     // hash table, or the two key buffers and counters of the sort
    int64_t scratch_entries;         // 8-byte entries available there
    int32_t id_bits;                 // bits of a node id (sort passes)
};

// Launch with programmatic stream serialization (the kernel starts with chain_wait()).
template <typename... KArgs, typename... Args>
inline cudaError_t launch_chained(void (*kernel)(KArgs...), int64_t grid, int block, cudaStream_t s, Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = dim3((unsigned)grid);
    cfg.blockDim = dim3((unsigned)block);
    cfg.dynamicSmemBytes = 0;
    cfg.stream = s;
    cudaLaunchAttribute at[1];
    at[0].id = cudaLaunchAttributeProgrammaticStreamSerialization;
    at[0].val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = at;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

void count_launches(int n);
// Streaming multiprocessors of the current device (looked up once per device).
int64_t sm_count();
// Grid size after the test knob gs_debug_set_grid_cap (0 = no cap) has been applied.
int64_t limit_grid(int64_t blocks);

// Caller-owned output buffers that replace the output regions of the workspace (used by the
// entry point whose scratch is a static device array).  Arrays are indexed by layer.
struct OutputBuffers {
    int32_t* input_nodes;
    int64_t input_nodes_capacity;
    int32_t* indptr[GS_MAX_HOPS];
    int64_t indptr_capacity[GS_MAX_HOPS];
    int32_t* indices[GS_MAX_HOPS];
    int64_t indices_capacity[GS_MAX_HOPS];
};

// Argument checks + one batch; `out` may be NULL (outputs then live in the workspace).
gs_status sample_batch_checked(gs_cache* c, const int32_t* d_seeds, int32_t num_seeds, gs_mode mode, double gamma,
                               uint32_t step, void* d_workspace, size_t workspace_bytes, cudaStream_t s,
                               gs_block* blocks, const int32_t** d_input_nodes, const int32_t** d_num_input_nodes,
                               const OutputBuffers* out);
gs_status set_error(gs_status code, const char* fmt, ...);
int32_t cache_num_hops(const gs_cache* c);
// Scratch bytes a batch of num_seeds seeds on this cache needs (what gs_workspace_bytes reports).
gs_status cache_workspace_bytes(const gs_cache* c, int32_t num_seeds, size_t* bytes);
// Looks up (and thereby materialises) the built-in scratch array of gs_sample_batch_noalloc on the current device.
gs_status prepare_noalloc_scratch();

cudaError_t launch_row_counts(const CountParams& p, int64_t n_bound, cudaStream_t s);
cudaError_t launch_refresh_pick(const StepParams& p, int64_t n_bound, cudaStream_t s);
cudaError_t launch_init_low_rows(const GraphView& g, int32_t* slots, int32_t pitch, int32_t W, int32_t caches,
                                 cudaStream_t s);
cudaError_t launch_scan(const StepParams& p, int64_t item_bound, cudaStream_t s);
cudaError_t launch_finish(const StepParams& p, int64_t n_bound, cudaStream_t s);
cudaError_t launch_relabel(const RelabelParams& p, int64_t n_bound, int64_t m_bound, cudaStream_t s);
// Pre-passes of the alternative dedup methods: both leave in aux[e] what the first-occurrence kernel needs
// (DEDUP_HASH: the table slot of the pick's id; DEDUP_SORT: the first position of the pick's id).
cudaError_t launch_dedup_hash(const RelabelParams& p, int64_t n_bound, int64_t m_bound, cudaStream_t s);
cudaError_t launch_dedup_sort(const RelabelParams& p, int64_t n_bound, int64_t m_bound, cudaStream_t s);
cudaError_t launch_gather(const void* src, int64_t src_ld_bytes, int64_t row_bytes, const int32_t* ids,
                          const int32_t* d_count, int32_t count_bound, void* dst, int64_t dst_ld_bytes,
                          int32_t blocks_per_sm /* 0: the default */, int64_t id_lo, int64_t id_hi /* ids outside
                          [id_lo, id_hi) are skipped */, cudaStream_t s);
cudaError_t gather_gave_up(cudaStream_t s, int* h_flag);
cudaError_t launch_gather_sharded(const void* const* bases, int32_t world, int64_t num_rows, int64_t rows_per_shard,
                                  int64_t src_ld_bytes,
                                  int64_t row_bytes, const int32_t* ids, const int32_t* d_count, int32_t count_bound,
                                  void* dst, int64_t dst_ld_bytes, cudaStream_t s);
cudaError_t launch_validate_graph(const GraphView& g, int64_t num_edges, int64_t* h_first_bad_row, cudaStream_t s);
cudaError_t launch_count_dense(const GraphView& g, int32_t theta, int64_t* h_count, cudaStream_t s);
cudaError_t launch_read_rows(const int32_t* slots, const int32_t* row_index, int32_t pitch, int32_t W,
                             const int32_t* nodes, int32_t n, int32_t* out, cudaStream_t s);
cudaError_t launch_shard_bucket(const int32_t* nodes, int32_t n, const int32_t* d_n, int32_t rows_per_shard, int32_t world,
                                int32_t capacity, int32_t* sorted, int32_t* slot, int32_t* counts_and_scratch, int32_t* status,
                                cudaStream_t s);
cudaError_t launch_export_picks(const int32_t* blk_indptr, const int32_t* picked, int32_t n, const int32_t* d_n, int32_t f,
                                int32_t* out, cudaStream_t s);
cudaError_t launch_import_picks(const int32_t* hdr, int32_t k, int32_t n_bound, int32_t f, const int32_t* reply,
                                int32_t reply_rows, const int32_t* slot, const int32_t* blk_indptr, int32_t* picked, unsigned long long* table,
                                uint32_t stamp, int64_t num_nodes, int32_t* status, cudaStream_t s);
cudaError_t launch_shard_merge(const int32_t* lists, const int32_t* counts, int32_t world, int32_t capacity, int64_t first_row,
                               int64_t rows_owned, int32_t* index, int32_t* distinct, int32_t* out_words, cudaStream_t s);
cudaError_t launch_shard_fan_out(const int32_t* lists, const int32_t* counts, int32_t world, int32_t capacity, int64_t first_row,
                                 int64_t rows_owned, int32_t* index, const int32_t* distinct, int32_t distinct_bound,
                                 const int32_t* rows, const int32_t* d_num_rows, int32_t f, int32_t* out, cudaStream_t s);
cudaError_t launch_build_row_index(const GraphView& g, int32_t theta, int32_t* row_index, int32_t* tile_sums,
                                   int32_t* d_dense_rows, cudaStream_t s);

}  // namespace gs
