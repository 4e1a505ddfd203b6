// S5 feature gather: out[p, :] = X[ids[p], :], a pure copy bound by HBM bandwidth.
//
// Rows are moved in the widest unit (16, 8, 4 or 2 bytes) that divides the row size, both row
// pitches and both base addresses.  A block covers `rows_per_iter` rows at a time, a fixed group
// of threads per row.  Measured on B200: full occupancy (8 blocks of 256 threads per SM, <= 32
// registers) with one or two rows in flight per thread beats fewer, fatter threads (83 % vs 70 %
// of the copy rate on 256-byte rows).  Loads and stores are marked streaming: no row is read twice
// (frontier ids are distinct).
#include "gs_device.cuh"
#include "gs_internal.h"

namespace gs {

#ifndef GS_GATHER_UNROLL
#define GS_GATHER_UNROLL 1
#endif
#ifndef GS_GATHER_MIN_BLOCKS
#define GS_GATHER_MIN_BLOCKS 8
#endif
// Blocks per SM in the grid (default; gs_graph_set_gather_grid overrides it per graph): 8 are
// resident, the rest queue behind them.  A few long-lived blocks are best when the gather has the GPU
// to itself (16 per SM: 0.193 ms for 2 M rows of 256 bytes; 256: 0.205; 1024: 0.248); many short
// blocks let the small kernels of a concurrent, higher-priority stream get SM slots within
// microseconds instead of after half the gather.
#ifndef GS_GATHER_GRID_PER_SM
#define GS_GATHER_GRID_PER_SM 256
#endif
constexpr int GT = 256;
constexpr int G_UNROLL = GS_GATHER_UNROLL;

template <typename V> __device__ __forceinline__ V ld_stream(const V* p) { return __ldcs(p); }
template <typename V> __device__ __forceinline__ void st_stream(V* p, V v) { __stcs(p, v); }

template <typename V>
__global__ void __launch_bounds__(GT, GS_GATHER_MIN_BLOCKS) k_gather(const char* __restrict__ src, int64_t src_ld, int units,
                                               const int32_t* __restrict__ ids, const int32_t* __restrict__ d_count,
                                               int count_bound, char* __restrict__ dst, int64_t dst_ld, int id_lo,
                                               int id_hi) {
    int n = d_count ? __ldg(d_count) : count_bound;
    if (n > count_bound) n = count_bound;
    // thread -> (row within group, first unit); tpr threads per row
    const int tpr = units < GT ? units : GT;
    const int rows_per_iter = GT / tpr;
    const int r_in = threadIdx.x / tpr;
    const int u0 = threadIdx.x - r_in * tpr;
    if (r_in >= rows_per_iter) return;
    const int64_t stride = (int64_t)gridDim.x * rows_per_iter;
    for (int64_t row = (int64_t)blockIdx.x * rows_per_iter + r_in; row < n; row += stride * G_UNROLL) {
        const V* s[G_UNROLL];
        V* d[G_UNROLL];
#pragma unroll
        for (int j = 0; j < G_UNROLL; ++j) {
            const int64_t rj = row + j * stride;
            const int32_t id = rj < n ? __ldg(ids + rj) : -1;
            // an id outside the rows the source holds is skipped: its output row is left as it is
            s[j] = (id >= id_lo && id < id_hi) ? reinterpret_cast<const V*>(src + (int64_t)id * src_ld) : nullptr;
            d[j] = reinterpret_cast<V*>(dst + rj * dst_ld);
        }
        for (int u = u0; u < units; u += tpr) {
            V val[G_UNROLL];
#pragma unroll
            for (int j = 0; j < G_UNROLL; ++j)
                if (s[j]) val[j] = ld_stream(s[j] + u);
#pragma unroll
            for (int j = 0; j < G_UNROLL; ++j)
                if (s[j]) st_stream(d[j] + u, val[j]);
        }
    }
}

// The same copy with the source split over several shards (row blocks of rows_per_shard rows, one
// base pointer each, possibly memory of peer GPUs mapped into this process): row `id` lives in
// shard id / rows_per_shard.  Plain streaming loads, so a remote row crosses NVLink exactly once
// and lands directly in the output: gather and transfer are one kernel, no staging buffer.
constexpr int GATHER_MAX_SHARDS = 64;
struct ShardBases {
    const char* base[GATHER_MAX_SHARDS];
};

template <typename V>
__global__ void __launch_bounds__(GT, GS_GATHER_MIN_BLOCKS) k_gather_sharded(const __grid_constant__ ShardBases shards,
                                                       int num_rows, int rows_per_shard, int64_t src_ld, int units,
                                                       const int32_t* __restrict__ ids,
                                                       const int32_t* __restrict__ d_count, int count_bound,
                                                       char* __restrict__ dst, int64_t dst_ld) {
    int n = d_count ? __ldg(d_count) : count_bound;
    if (n > count_bound) n = count_bound;
    const int tpr = units < GT ? units : GT;
    const int rows_per_iter = GT / tpr;
    const int r_in = threadIdx.x / tpr;
    const int u0 = threadIdx.x - r_in * tpr;
    if (r_in >= rows_per_iter) return;
    const int64_t stride = (int64_t)gridDim.x * rows_per_iter;
    for (int64_t row = (int64_t)blockIdx.x * rows_per_iter + r_in; row < n; row += stride) {
        const int32_t id = __ldg(ids + row);
        if (id < 0 || id >= num_rows) continue;   // not a row of the matrix: the output row is left untouched
        const int o = id / rows_per_shard;
        const V* s = reinterpret_cast<const V*>(shards.base[o] + (int64_t)(id - o * rows_per_shard) * src_ld);
        V* d = reinterpret_cast<V*>(dst + row * dst_ld);
        for (int u = u0; u < units; u += tpr) st_stream(d + u, ld_stream(s + u));
    }
}

template <typename V>
static void launch_sharded_t(const ShardBases& sh, int num_rows, int rows_per_shard, int64_t src_ld, int64_t row_bytes,
                             const int32_t* ids, const int32_t* d_count, int32_t count_bound, void* dst, int64_t dst_ld,
                             cudaStream_t s) {
    const int units = (int)(row_bytes / (int64_t)sizeof(V));
    const int tpr = units < GT ? units : GT;
    const int rows_per_iter = GT / tpr;
    int64_t blocks = ((int64_t)count_bound + rows_per_iter - 1) / rows_per_iter;
    const int64_t cap = sm_count() * GS_GATHER_GRID_PER_SM;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    k_gather_sharded<V><<<(int)blocks, GT, 0, s>>>(sh, num_rows, rows_per_shard, src_ld, units, ids, d_count, count_bound,
                                                  (char*)dst, dst_ld);
}

cudaError_t launch_gather_sharded(const void* const* bases, int32_t world, int64_t num_rows, int64_t rows_per_shard, int64_t src_ld_bytes,
                                  int64_t row_bytes, const int32_t* ids, const int32_t* d_count, int32_t count_bound,
                                  void* dst, int64_t dst_ld_bytes, cudaStream_t s) {
    if (count_bound <= 0 || row_bytes <= 0) return cudaSuccess;
    if (world < 1 || world > GATHER_MAX_SHARDS) return cudaErrorInvalidValue;
    ShardBases sh{};
    uint64_t all = (uint64_t)(uintptr_t)dst | (uint64_t)src_ld_bytes | (uint64_t)dst_ld_bytes | (uint64_t)row_bytes;
    for (int o = 0; o < world; ++o) {
        sh.base[o] = (const char*)bases[o];
        all |= (uint64_t)(uintptr_t)bases[o];
    }
    const int rps = (int)rows_per_shard;
    if ((all & 15) == 0) launch_sharded_t<uint4>(sh, (int)num_rows, rps, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, s);
    else if ((all & 7) == 0) launch_sharded_t<uint2>(sh, (int)num_rows, rps, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, s);
    else if ((all & 3) == 0) launch_sharded_t<uint32_t>(sh, (int)num_rows, rps, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, s);
    else launch_sharded_t<uint16_t>(sh, (int)num_rows, rps, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, s);
    count_launches(1);
    return cudaGetLastError();
}

template <typename V>
static void launch_t(const void* src, int64_t src_ld, int64_t row_bytes, const int32_t* ids, const int32_t* d_count,
                     int32_t count_bound, void* dst, int64_t dst_ld, int32_t blocks_per_sm, int id_lo, int id_hi,
                     cudaStream_t s) {
    const int units = (int)(row_bytes / (int64_t)sizeof(V));
    const int tpr = units < GT ? units : GT;
    const int rows_per_iter = GT / tpr;
    int64_t blocks = ((int64_t)count_bound + (int64_t)rows_per_iter * G_UNROLL - 1) / ((int64_t)rows_per_iter * G_UNROLL);
    const int64_t cap = sm_count() * (int64_t)(blocks_per_sm > 0 ? blocks_per_sm : GS_GATHER_GRID_PER_SM);
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    blocks = limit_grid(blocks);
    k_gather<V><<<(int)blocks, GT, 0, s>>>((const char*)src, src_ld, units, ids, d_count, count_bound, (char*)dst, dst_ld,
                                           id_lo, id_hi);
}

cudaError_t launch_gather(const void* src, int64_t src_ld_bytes, int64_t row_bytes, const int32_t* ids,
                          const int32_t* d_count, int32_t count_bound, void* dst, int64_t dst_ld_bytes,
                          int32_t blocks_per_sm, int64_t id_lo, int64_t id_hi, cudaStream_t s) {
    if (count_bound <= 0 || row_bytes <= 0) return cudaSuccess;
    if (id_lo < 0) id_lo = 0;
    if (id_hi > 0x7FFFFFFFll) id_hi = 0x7FFFFFFFll;
    const uint64_t all = (uint64_t)(uintptr_t)src | (uint64_t)(uintptr_t)dst | (uint64_t)src_ld_bytes |
                         (uint64_t)dst_ld_bytes | (uint64_t)row_bytes;
    if ((all & 15) == 0) launch_t<uint4>(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, blocks_per_sm, (int)id_lo, (int)id_hi, s);
    else if ((all & 7) == 0) launch_t<uint2>(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, blocks_per_sm, (int)id_lo, (int)id_hi, s);
    else if ((all & 3) == 0) launch_t<uint32_t>(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, blocks_per_sm, (int)id_lo, (int)id_hi, s);
    else launch_t<uint16_t>(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, blocks_per_sm, (int)id_lo, (int)id_hi, s);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace gs
