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
constexpr int HDR_WORDS = HDR_TICKET_E + GS_MAX_HOPS;
constexpr size_t HDR_BYTES = 1024;
static_assert(HDR_WORDS * 4 <= HDR_BYTES, "header too small");

constexpr int SCAN_A_TILE = 1024;  // frontier nodes per tile of the row-count scan
constexpr int SCAN_E_TILE = 4096;  // picked edges per tile of the first-occurrence scan

inline size_t align_up(size_t x, size_t a) { return (x + a - 1) / a * a; }

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
    size_t picked, aux, tiles_a, tiles_e, hub_list;
    size_t total;
};

inline WorkspaceLayout make_layout(const Bounds& b) {
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
    w.hub_list = take((size_t)max_n * 4);
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
    int32_t* slots;        // this step's cache: [num_nodes][pitch]
    int32_t pitch, W, f, r;
    uint32_t step, key0, key1;
    uint32_t word_fill, word_evict, word_pick;  // (purpose << 8) | tag
    const int32_t* frontier;     // NULL: identity (node id = position)
    const int32_t* d_n;          // device count of frontier nodes, or NULL -> n_host
    int32_t n_host;
    const int32_t* d_refresh_from;  // device scalar: positions below it are not refreshed; NULL -> 0
    const int32_t* blk_indptr;   // final offsets of each node's picks
    int32_t* picked;             // global ids of the picks
    unsigned long long* table;   // relabel table, (stamp << 32) | position
    uint32_t stamp;
    int32_t n_base_is_device;    // position of pick e in the concatenated list is *d_n + e
    int32_t* hub_list;
    int32_t* hub_count;
    int32_t* work_counter;
    int32_t* status;
    int32_t do_pick, init_rows;
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
};

struct RelabelParams {
    int32_t* hdr;
    int32_t k;
    const int32_t* picked;
    int32_t* aux;
    int32_t* tile_sums;
    int32_t* frontier;
    int32_t* local;
    unsigned long long* table;
    uint32_t stamp;
    int64_t n_cap;
};

void count_launches(int n);

cudaError_t launch_row_counts(const CountParams& p, int64_t n_bound, cudaStream_t s);
cudaError_t launch_refresh_pick(const StepParams& p, int64_t n_bound, cudaStream_t s);
cudaError_t launch_relabel(const RelabelParams& p, int64_t m_bound, cudaStream_t s);
cudaError_t launch_gather(const void* src, int64_t src_ld_bytes, int64_t row_bytes, const int32_t* ids,
                          const int32_t* d_count, int32_t count_bound, void* dst, int64_t dst_ld_bytes,
                          cudaStream_t s);
cudaError_t launch_read_rows(const int32_t* slots, int32_t pitch, int32_t W, const int32_t* nodes, int32_t n,
                             int32_t* out, cudaStream_t s);

}  // namespace gs
