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
    if (d_n) n = min(n, max(0, __ldcg(d_n)));   // the list's length may live on the device; n is its bound then
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
                                                                int world, const int32_t* __restrict__ counts,
                                                                int32_t* __restrict__ cursor, int32_t* __restrict__ sorted,
                                                                int32_t* __restrict__ slot) {
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
    if (threadIdx.x < world) {
        int start = 0;
        for (int j = 0; j < (int)threadIdx.x; ++j) start += __ldg(counts + j);
        base[threadIdx.x] = start + (hist[threadIdx.x] ? atomicAdd(cursor + threadIdx.x, hist[threadIdx.x]) : 0);
    }
    __syncthreads();
    if (i < n) {
        const int pos = o >= 0 ? base[o] + rank : -1;
        slot[i] = pos;
        if (pos >= 0) sorted[pos] = v;
    }
}

cudaError_t launch_shard_bucket(const int32_t* nodes, int32_t n, const int32_t* d_n, int32_t rows_per_shard, int32_t world, int32_t* sorted,
                                int32_t* slot, int32_t* counts_and_scratch, int32_t* status, cudaStream_t s) {
    cudaError_t e = cudaMemsetAsync(counts_and_scratch, 0, (size_t)(2 * world + 1) * sizeof(int32_t), s);
    if (e != cudaSuccess || n <= 0) return e;
    const int blocks = (n + SHARD_THREADS - 1) / SHARD_THREADS;
    k_bucket_count<<<blocks, SHARD_THREADS, 0, s>>>(nodes, n, d_n, rows_per_shard, world, counts_and_scratch, status);
    k_bucket_place<<<blocks, SHARD_THREADS, 0, s>>>(nodes, n, d_n, rows_per_shard, world, counts_and_scratch,
                                                    counts_and_scratch + world, sorted, slot);
    count_launches(2);
    return cudaGetLastError();
}

// Owner side: the picks of node p, picked[blk_indptr[p] .. blk_indptr[p+1]), as a fixed row of f ids.
__global__ void __launch_bounds__(SHARD_THREADS) k_export_picks(const int32_t* __restrict__ blk_indptr,
                                                                const int32_t* __restrict__ picked, int n, int f,
                                                                int32_t* __restrict__ out) {
    const int64_t i = (int64_t)blockIdx.x * SHARD_THREADS + threadIdx.x;
    if (i >= (int64_t)n * f) return;
    const int p = (int)(i / f), t = (int)(i - (int64_t)p * f);
    const int lo = __ldg(blk_indptr + p), hi = __ldg(blk_indptr + p + 1);
    out[i] = (lo + t < hi) ? __ldg(picked + lo + t) : -1;
}

cudaError_t launch_export_picks(const int32_t* blk_indptr, const int32_t* picked, int32_t n, int32_t f, int32_t* out,
                                cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const int64_t blocks = ((int64_t)n * f + SHARD_THREADS - 1) / SHARD_THREADS;
    k_export_picks<<<(unsigned)blocks, SHARD_THREADS, 0, s>>>(blk_indptr, picked, n, f, out);
    count_launches(1);
    return cudaGetLastError();
}

// Requester side: the returned rows become the step's picked-edge array, and every pick claims its
// id in the relabel table with its edge position - what the pick kernels do when they run locally.
__global__ void __launch_bounds__(SHARD_THREADS) k_import_picks(const int32_t* __restrict__ hdr, int k, int f,
                                                                const int32_t* __restrict__ reply,
                                                                const int32_t* __restrict__ slot,
                                                                const int32_t* __restrict__ blk_indptr,
                                                                int32_t* __restrict__ picked, unsigned long long* table,
                                                                uint32_t stamp, int64_t num_nodes, int32_t* status) {
    if (__ldcg(hdr + HDR_STATUS) != 0) return;
    const int n = __ldcg(hdr + HDR_N + k);
    const int64_t i = (int64_t)blockIdx.x * SHARD_THREADS + threadIdx.x;
    if (i >= (int64_t)n * f) return;
    const int p = (int)(i / f), t = (int)(i - (int64_t)p * f);
    const int sl = slot ? __ldg(slot + p) : p;
    if ((unsigned)sl >= (unsigned)n) return;      // reported by the row-count kernel; the row has no picks
    const int32_t u = __ldg(reply + (int64_t)sl * f + t);
    if (u < 0) return;
    if ((int64_t)u >= num_nodes) {
        atomicCAS(status, 0, GS_ERR_RANGE);
        return;
    }
    const int e = __ldg(blk_indptr + p) + t;
    if (e >= __ldg(blk_indptr + p + 1)) return;   // beyond the row's non-negative prefix: not a pick
    picked[e] = u;
    atomicMin(table + u, ((unsigned long long)stamp << 32) | ((uint32_t)n + (uint32_t)e));
}

cudaError_t launch_import_picks(const int32_t* hdr, int32_t k, int32_t n_bound, int32_t f, const int32_t* reply,
                                const int32_t* slot, const int32_t* blk_indptr, int32_t* picked, unsigned long long* table,
                                uint32_t stamp, int64_t num_nodes, int32_t* status, cudaStream_t s) {
    if (n_bound <= 0) return cudaSuccess;
    const int64_t blocks = ((int64_t)n_bound * f + SHARD_THREADS - 1) / SHARD_THREADS;
    k_import_picks<<<(unsigned)blocks, SHARD_THREADS, 0, s>>>(hdr, k, f, reply, slot, blk_indptr, picked, table, stamp,
                                                              num_nodes, status);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace gs
