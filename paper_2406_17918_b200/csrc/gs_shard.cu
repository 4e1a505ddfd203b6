// Node-sharded sampling: the kernels around the per-hop exchange.
//
// Nodes are partitioned by id range, shard o owns [o * rows_per_shard, (o + 1) * rows_per_shard).
// A hop of one rank's batch is: bucket the frontier by owner, send each owner its nodes, the
// owners refresh and pick (the ordinary scan / finish kernels, their picks exported as fixed
// rows of f ids), the rows come back, and the requester turns them into the picked-edge array
// and the relabel-table claims that the ordinary kernels would have produced locally.  Every
// random choice is keyed by (seed, node, item, step), so the result does not depend on which
// device evaluates it.  Nothing here waits on another block or another device.
#include "gs_device.cuh"
#include "gs_internal.h"

namespace gs {

constexpr int SHARD_THREADS = 256;
constexpr int SHARD_MAX_WORLD = 64;

// Pass 1: how many of the n nodes belong to each owner (block-local histogram, one global atomic
// per owner and block).
__global__ void __launch_bounds__(SHARD_THREADS) k_bucket_count(const int32_t* __restrict__ nodes, int n, const int32_t* __restrict__ d_n,
                                                                int rows_per_shard,
                                                                int world, int32_t* __restrict__ counts, int32_t* status) {
    __shared__ int hist[SHARD_MAX_WORLD];
    if (d_n) {   // the list's length may live on the device; n is its bound then, and a longer list is an error
        const int len = __ldcg(d_n);
        if (len > n && blockIdx.x == 0 && threadIdx.x == 0) atomicCAS(status, 0, GS_ERR_WORKSPACE);
        n = min(n, max(0, len));
    }
    if (threadIdx.x < SHARD_MAX_WORLD) hist[threadIdx.x] = 0;
    __syncthreads();
    const int i = blockIdx.x * SHARD_THREADS + threadIdx.x;
    if (i < n) {
        const int32_t v = __ldg(nodes + i);
        const int o = v >= 0 ? v / rows_per_shard : world;
        if (o >= world) atomicCAS(status, 0, GS_ERR_RANGE);
        else atomicAdd(&hist[o], 1);
    }
    __syncthreads();
    if (threadIdx.x < world && hist[threadIdx.x]) atomicAdd(counts + threadIdx.x, hist[threadIdx.x]);
}

// Pass 2: place every node in its owner's segment of `sorted` and remember where it went.  The
// order inside a segment is whatever the atomics give; `slot` is what ties a reply to its node.
__global__ void __launch_bounds__(SHARD_THREADS) k_bucket_place(const int32_t* __restrict__ nodes, int n, const int32_t* __restrict__ d_n,
                                                                int rows_per_shard,
                                                                int world, int capacity, const int32_t* __restrict__ counts,
                                                                int32_t* __restrict__ cursor, int32_t* __restrict__ sorted,
                                                                int32_t* __restrict__ slot, int32_t* status) {
    __shared__ int hist[SHARD_MAX_WORLD];
    __shared__ int base[SHARD_MAX_WORLD];
    if (d_n) n = min(n, max(0, __ldcg(d_n)));
    if (threadIdx.x < SHARD_MAX_WORLD) hist[threadIdx.x] = 0;
    __syncthreads();
    const int i = blockIdx.x * SHARD_THREADS + threadIdx.x;
    int32_t v = -1;
    int o = -1, rank = 0;
    if (i < n) {
        v = __ldg(nodes + i);
        o = v >= 0 ? v / rows_per_shard : world;
        if (o >= world) o = -1;
        else rank = atomicAdd(&hist[o], 1);
    }
    __syncthreads();
    // packed: owner o's segment starts where the smaller owners' end; fixed pitch: at o * capacity, and a
    // node beyond the segment's capacity is dropped and reported
    if (threadIdx.x < world) {
        int start = 0;
        if (capacity > 0) start = (int)threadIdx.x * capacity;
        else
            for (int j = 0; j < (int)threadIdx.x; ++j) start += __ldg(counts + j);
        base[threadIdx.x] = (hist[threadIdx.x] ? atomicAdd(cursor + threadIdx.x, hist[threadIdx.x]) : 0);
        hist[threadIdx.x] = start;   // every rank of this block was taken before the barrier above
    }
    __syncthreads();
    if (i < n) {
        int pos = -1;
        if (o >= 0) {
            const int in_segment = base[o] + rank;
            if (capacity > 0 && in_segment >= capacity) atomicCAS(status, 0, GS_ERR_WORKSPACE);
            else pos = hist[o] + in_segment;
        }
        slot[i] = pos;
        if (pos >= 0) sorted[pos] = v;
    }
}

cudaError_t launch_shard_bucket(const int32_t* nodes, int32_t n, const int32_t* d_n, int32_t rows_per_shard, int32_t world,
                                int32_t capacity, int32_t* sorted, int32_t* slot, int32_t* counts_and_scratch, int32_t* status,
                                cudaStream_t s) {
    cudaError_t e = cudaMemsetAsync(counts_and_scratch, 0, (size_t)(2 * world + 1) * sizeof(int32_t), s);
    if (e != cudaSuccess || n <= 0) return e;
    const int blocks = (n + SHARD_THREADS - 1) / SHARD_THREADS;
    k_bucket_count<<<blocks, SHARD_THREADS, 0, s>>>(nodes, n, d_n, rows_per_shard, world, counts_and_scratch, status);
    k_bucket_place<<<blocks, SHARD_THREADS, 0, s>>>(nodes, n, d_n, rows_per_shard, world, capacity, counts_and_scratch,
                                                    counts_and_scratch + world, sorted, slot, status);
    count_launches(2);
    return cudaGetLastError();
}

// Both pick-row kernels walk (node, item) pairs with a capped grid: the host only knows an upper bound of the
// list's length, often several times the real one, and a block per 256 pairs of the bound costs more than the copy.
__device__ __forceinline__ void split_pair(unsigned long long i, unsigned f, unsigned& p, unsigned& t) {
    p = (i >> 32) ? (unsigned)(i / f) : (unsigned)i / f;
    t = (unsigned)(i - (unsigned long long)p * f);
}

// Owner side: the picks of node p, picked[blk_indptr[p] .. blk_indptr[p+1]), as a fixed row of f ids.
__global__ void __launch_bounds__(SHARD_THREADS) k_export_picks(const int32_t* __restrict__ blk_indptr,
                                                                const int32_t* __restrict__ picked, int n,
                                                                const int32_t* __restrict__ d_n, int f,
                                                                int32_t* __restrict__ out) {
    n = min(n, max(0, __ldcg(d_n)));   // rows of the list that were sampled (none after a device-detected error)
    const unsigned long long total = (unsigned long long)n * (unsigned)f;
    for (unsigned long long i = (unsigned long long)blockIdx.x * SHARD_THREADS + threadIdx.x; i < total;
         i += (unsigned long long)gridDim.x * SHARD_THREADS) {
        unsigned p, t;
        split_pair(i, (unsigned)f, p, t);
        const int lo = __ldg(blk_indptr + p), hi = __ldg(blk_indptr + p + 1);
        out[i] = (lo + (int)t < hi) ? __ldg(picked + lo + t) : -1;
    }
}

static unsigned pair_grid(int64_t n_bound, int32_t f) {
    int64_t blocks = (n_bound * f + SHARD_THREADS - 1) / SHARD_THREADS;
    const int64_t cap = sm_count() * 16;
    return (unsigned)limit_grid(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
}

cudaError_t launch_export_picks(const int32_t* blk_indptr, const int32_t* picked, int32_t n, const int32_t* d_n, int32_t f,
                                int32_t* out, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    k_export_picks<<<pair_grid(n, f), SHARD_THREADS, 0, s>>>(blk_indptr, picked, n, d_n, f, out);
    count_launches(1);
    return cudaGetLastError();
}

// Requester side: the returned rows become the step's picked-edge array, and (with the direct-address
// table; `table` is NULL otherwise) every pick claims its id in the relabel table with its edge
// position - what the pick kernels do when they run locally.
__global__ void __launch_bounds__(SHARD_THREADS) k_import_picks(const int32_t* __restrict__ hdr, int k, int f,
                                                                const int32_t* __restrict__ reply, int reply_rows,
                                                                const int32_t* __restrict__ slot,
                                                                const int32_t* __restrict__ blk_indptr,
                                                                int32_t* __restrict__ picked, unsigned long long* table,
                                                                uint32_t stamp, int64_t num_nodes, int32_t* status) {
    if (__ldcg(hdr + HDR_STATUS) != 0) return;
    const int n = __ldcg(hdr + HDR_N + k);
    const unsigned rows = (unsigned)(reply_rows > 0 ? reply_rows : n);
    const unsigned long long total = (unsigned long long)max(n, 0) * (unsigned)f;
    for (unsigned long long i = (unsigned long long)blockIdx.x * SHARD_THREADS + threadIdx.x; i < total;
         i += (unsigned long long)gridDim.x * SHARD_THREADS) {
        unsigned p, t;
        split_pair(i, (unsigned)f, p, t);
        const int sl = slot ? __ldg(slot + p) : (int)p;
        if ((unsigned)sl >= rows) continue;           // reported by the row-count kernel; the row has no picks
        const int32_t u = __ldg(reply + (int64_t)sl * f + t);
        if (u < 0) continue;
        if ((int64_t)u >= num_nodes) {
            atomicCAS(status, 0, GS_ERR_RANGE);
            continue;
        }
        const int e = __ldg(blk_indptr + p) + (int)t;
        if (e >= __ldg(blk_indptr + p + 1)) continue;   // beyond the row's non-negative prefix: not a pick
        picked[e] = u;
        if (table) atomicMin(table + u, ((unsigned long long)stamp << 32) | ((uint32_t)n + (uint32_t)e));
    }
}

cudaError_t launch_import_picks(const int32_t* hdr, int32_t k, int32_t n_bound, int32_t f, const int32_t* reply,
                                int32_t reply_rows, const int32_t* slot, const int32_t* blk_indptr, int32_t* picked, unsigned long long* table,
                                uint32_t stamp, int64_t num_nodes, int32_t* status, cudaStream_t s) {
    if (n_bound <= 0) return cudaSuccess;
    k_import_picks<<<pair_grid(n_bound, f), SHARD_THREADS, 0, s>>>(hdr, k, f, reply, reply_rows, slot, blk_indptr, picked, table,
                                                                   stamp, num_nodes, status);
    count_launches(1);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- owner side: all requesters' lists at once
// A hub sits in every requester's frontier, and serving the lists one by one scans its row once per requester.
// The lists (fixed pitch, lengths on the device) are merged instead: every owned node that anyone asks for
// gets one position in a list of distinct nodes (`index`, one word per owned row, -1 = not asked for), that
// list is sampled once, and the rows are fanned out to the requesters' segments.  Same rows either way:
// picks are keyed by (node, step), not by who asks.
__global__ void __launch_bounds__(SHARD_THREADS) k_merge_claim(const int32_t* __restrict__ lists,
                                                               const int32_t* __restrict__ counts, int world, int capacity,
                                                               int64_t first_row, int64_t rows_owned, int32_t* index,
                                                               int32_t* __restrict__ distinct, int32_t* out_words) {
    __shared__ int s_new, s_base;
    const int64_t total = (int64_t)world * capacity;
    for (int64_t e0 = (int64_t)blockIdx.x * SHARD_THREADS; e0 < total; e0 += (int64_t)gridDim.x * SHARD_THREADS) {
        if (threadIdx.x == 0) s_new = 0;
        __syncthreads();
        const int64_t e = e0 + threadIdx.x;
        int32_t v = -1;
        int64_t loc = -1;
        int rank = -1;
        if (e < total) {
            const int r = (int)(e / capacity), i = (int)(e - (int64_t)r * capacity);
            if (i < min(max(__ldg(counts + r), 0), capacity)) {
                v = __ldg(lists + e);
                loc = (int64_t)v - first_row;
                if (loc < 0 || loc >= rows_owned) {
                    atomicCAS(out_words + 1, 0, GS_ERR_RANGE);
                    loc = -1;
                } else if (atomicCAS(index + loc, -1, -2) == -1) {
                    rank = atomicAdd(&s_new, 1);          // the first to ask for this node places it
                }
            }
        }
        __syncthreads();
        if (threadIdx.x == 0) s_base = s_new ? atomicAdd(out_words, s_new) : 0;
        __syncthreads();
        if (rank >= 0) {
            distinct[s_base + rank] = v;
            index[loc] = s_base + rank;
        }
        __syncthreads();   // s_new and s_base are reused by the next round
    }
}

// out[e][:] = rows[index[node of entry e]][:] for every entry of every requester's list.
__global__ void __launch_bounds__(SHARD_THREADS) k_fan_out(const int32_t* __restrict__ lists, const int32_t* __restrict__ counts,
                                                           int world, int capacity, int64_t first_row, int64_t rows_owned,
                                                           const int32_t* __restrict__ index, const int32_t* __restrict__ rows,
                                                           const int32_t* __restrict__ d_num_rows, int f,
                                                           int32_t* __restrict__ out) {
    const int num_rows = __ldcg(d_num_rows);
    const unsigned long long total = (unsigned long long)world * capacity * (unsigned)f;
    for (unsigned long long i = (unsigned long long)blockIdx.x * SHARD_THREADS + threadIdx.x; i < total;
         i += (unsigned long long)gridDim.x * SHARD_THREADS) {
        unsigned e, t;
        split_pair(i, (unsigned)f, e, t);
        const unsigned r = e / (unsigned)capacity, j = e - r * (unsigned)capacity;
        if ((int)j >= min(max(__ldg(counts + r), 0), capacity)) continue;
        const int64_t loc = (int64_t)__ldg(lists + e) - first_row;
        if (loc < 0 || loc >= rows_owned) continue;        // reported by the merge
        const int pos = __ldcg(index + loc);
        out[i] = ((unsigned)pos < (unsigned)num_rows) ? __ldg(rows + (int64_t)pos * f + t) : -1;
    }
}

// The index goes back to "nobody asks" for exactly the nodes that were placed.
__global__ void __launch_bounds__(SHARD_THREADS) k_merge_reset(const int32_t* __restrict__ distinct,
                                                               const int32_t* __restrict__ d_num, int bound, int64_t first_row,
                                                               int64_t rows_owned, int32_t* index) {
    const int n = min(bound, max(0, __ldcg(d_num)));
    for (int j = blockIdx.x * SHARD_THREADS + threadIdx.x; j < n; j += gridDim.x * SHARD_THREADS) {
        const int64_t loc = (int64_t)__ldg(distinct + j) - first_row;
        if (loc >= 0 && loc < rows_owned) index[loc] = -1;
    }
}

cudaError_t launch_shard_merge(const int32_t* lists, const int32_t* counts, int32_t world, int32_t capacity, int64_t first_row,
                               int64_t rows_owned, int32_t* index, int32_t* distinct, int32_t* out_words, cudaStream_t s) {
    cudaError_t e = cudaMemsetAsync(out_words, 0, 2 * sizeof(int32_t), s);
    if (e != cudaSuccess) return e;
    int64_t blocks = ((int64_t)world * capacity + SHARD_THREADS - 1) / SHARD_THREADS;
    const int64_t cap = sm_count() * 16;
    blocks = limit_grid(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
    k_merge_claim<<<(unsigned)blocks, SHARD_THREADS, 0, s>>>(lists, counts, world, capacity, first_row, rows_owned, index,
                                                             distinct, out_words);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_shard_fan_out(const int32_t* lists, const int32_t* counts, int32_t world, int32_t capacity, int64_t first_row,
                                 int64_t rows_owned, int32_t* index, const int32_t* distinct, int32_t distinct_bound,
                                 const int32_t* rows, const int32_t* d_num_rows, int32_t f, int32_t* out, cudaStream_t s) {
    k_fan_out<<<pair_grid((int64_t)world * capacity, f), SHARD_THREADS, 0, s>>>(lists, counts, world, capacity, first_row,
                                                                               rows_owned, index, rows, d_num_rows, f, out);
    int64_t blocks = ((int64_t)distinct_bound + SHARD_THREADS - 1) / SHARD_THREADS;
    const int64_t cap = sm_count() * 16;
    blocks = limit_grid(blocks < cap ? (blocks < 1 ? 1 : blocks) : cap);
    k_merge_reset<<<(unsigned)blocks, SHARD_THREADS, 0, s>>>(distinct, d_num_rows, distinct_bound, first_row, rows_owned, index);
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace gs
