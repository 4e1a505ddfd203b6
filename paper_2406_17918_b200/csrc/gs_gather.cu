// S5 feature gather: out[p, :] = X[ids[p], :], a pure copy bound by HBM bandwidth.
//
// Two kernels.  k_gather_bulk (the default for rows of 128 to 512 bytes on 64-byte boundaries) lets the SM's
// copy engine move the rows: bulk copies global -> shared memory -> global, a lane per row, nothing held in
// registers - 0.90 of the measured copy rate on 256-byte rows.  k_gather<V> moves rows in the widest unit (16,
// 8, 4 or 2 bytes) that divides the row size, both row pitches and both base addresses, a fixed group of threads
// per row; measured on B200: full occupancy (8 blocks of 256 threads per SM, <= 32 registers) with one or two
// rows in flight per thread beats fewer, fatter threads (0.82 vs 0.70 of the copy rate on 256-byte rows).  It
// serves every other row shape, and the many-short-blocks launch shape a gather beside another stream wants.
// Loads and stores are marked streaming: no row is read twice (frontier ids are distinct).
#include <atomic>

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

// ---------------------------------------------------------------- bulk-copy variant
// The same copy with the rows moved by the copy engine of the SM instead of by loads and stores: a lane asks for
// its row with one bulk copy (global -> shared memory, completion counted on an mbarrier), waits for the warp's 32
// rows and writes its row out with a second bulk copy (shared -> global).  A warp owns BULK_STAGES slices of 32
// rows in shared memory, so rows are in flight without a register being held for them.  Needs 16-byte aligned rows
// on both sides (the launch asks for 64) and rows of at most BULK_MAX_ROW bytes; every wait on a barrier is bounded (a warp that gives up
// sets g_gather_gave_up, which gs_gather_status reports).
#ifndef GS_BULK_WARPS
#define GS_BULK_WARPS 4
#endif
#ifndef GS_BULK_STAGES
#define GS_BULK_STAGES 2
#endif
constexpr int BULK_WARPS = GS_BULK_WARPS;
constexpr int BULK_STAGES = GS_BULK_STAGES;
constexpr int BULK_MIN_ROW = 128;
constexpr int BULK_MAX_ROW = 512;
constexpr unsigned BULK_WAIT_LIMIT = 1u << 22;   // polls of one mbarrier phase before the warp gives up

__device__ int g_gather_gave_up;   // set when a wait ran out

__device__ __forceinline__ uint32_t smem_u32(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__global__ void __launch_bounds__(BULK_WARPS * 32) k_gather_bulk(const char* __restrict__ src, int64_t src_ld, int row_bytes,
                                                                 const int32_t* __restrict__ ids,
                                                                 const int32_t* __restrict__ d_count, int count_bound,
                                                                 char* __restrict__ dst, int64_t dst_ld, int id_lo, int id_hi) {
    extern __shared__ __align__(128) unsigned char bulk_smem[];
    __shared__ __align__(8) unsigned long long bars[BULK_WARPS][BULK_STAGES];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    int n = d_count ? __ldg(d_count) : count_bound;
    if (n > count_bound) n = count_bound;
    unsigned char* mine = bulk_smem + (size_t)warp * BULK_STAGES * 32 * row_bytes;
    if (lane == 0) {
#pragma unroll
        for (int s = 0; s < BULK_STAGES; ++s)
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(smem_u32(&bars[warp][s])));
    }
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");   // the copy engine sees the initialised barriers
    __syncwarp();
    const long long groups = ((long long)n + 31) / 32;
    const int warps = blockDim.x >> 5;      // 1 .. BULK_WARPS, chosen by the launch so that the slices fit
    const long long first = (long long)blockIdx.x * warps + warp, step = (long long)gridDim.x * warps;
    bool ok[BULK_STAGES];
    long long row_of[BULK_STAGES];

    auto issue = [&](long long g, int s) {
        const long long row = g * 32 + lane;
        const int32_t id = row < n ? __ldg(ids + row) : -1;
        ok[s] = id >= id_lo && id < id_hi;     // an id outside the rows the source holds is skipped
        row_of[s] = row;
        const unsigned mask = __ballot_sync(FULL, ok[s]);
        const uint32_t bar = smem_u32(&bars[warp][s]);
        if (lane == 0)
            asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"((unsigned)__popc(mask) * row_bytes)
                         : "memory");
        __syncwarp();
        if (ok[s])
            asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
                             smem_u32(mine + ((size_t)s * 32 + lane) * row_bytes)),
                         "l"(src + (int64_t)id * src_ld), "r"(row_bytes), "r"(bar)
                         : "memory");
    };
    auto drain = [&](int s, unsigned parity) -> bool {
        const uint32_t bar = smem_u32(&bars[warp][s]);
        unsigned done = 0, polls = 0;
        while (!done && polls < BULK_WAIT_LIMIT) {
            asm volatile("{ .reg .pred p; mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2; selp.u32 %0, 1, 0, p; }"
                         : "=r"(done)
                         : "r"(bar), "r"(parity)
                         : "memory");
            ++polls;
        }
        if (!__all_sync(FULL, done != 0)) return false;
        asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
        if (ok[s])
            asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(dst + row_of[s] * dst_ld),
                         "r"(smem_u32(mine + ((size_t)s * 32 + lane) * row_bytes)), "r"(row_bytes)
                         : "memory");
        asm volatile("cp.async.bulk.commit_group;" ::: "memory");
        return true;
    };

    // software pipeline over the warp's groups: round `it` first writes out group it - (BULK_STAGES - 1), then asks
    // for group `it`, whose slice was last read by the store of round it - 1 - that store is the one before the
    // thread's latest, so it has left shared memory once at most one of the thread's store groups is pending
    long long it = 0;
    bool fine = true;
    for (long long g = first; g < groups && fine; g += step, ++it) {
        if (it >= BULK_STAGES - 1) {
            const long long jt = it - (BULK_STAGES - 1);
            fine = drain((int)(jt % BULK_STAGES), (unsigned)((jt / BULK_STAGES) & 1));
            if (!fine) break;
        }
        if (it >= BULK_STAGES) asm volatile("cp.async.bulk.wait_group.read 1;" ::: "memory");
        issue(g, (int)(it % BULK_STAGES));
    }
    // the groups still in flight
    for (long long jt = it >= BULK_STAGES - 1 ? it - (BULK_STAGES - 1) : 0; jt < it && fine; ++jt)
        fine = drain((int)(jt % BULK_STAGES), (unsigned)((jt / BULK_STAGES) & 1));
    asm volatile("cp.async.bulk.wait_group 0;" ::: "memory");   // nothing of this thread is left in flight at exit
    if (!fine && lane == 0) atomicExch(&g_gather_gave_up, 1);
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

static cudaError_t launch_bulk(const void* src, int64_t src_ld, int64_t row_bytes, const int32_t* ids, const int32_t* d_count,
                               int32_t count_bound, void* dst, int64_t dst_ld, int id_lo, int id_hi, cudaStream_t s) {
    // up to 96 KB of slices per block (two blocks per SM): 4 warps for rows up to 384 bytes, 3 above
    int warps = (int)((96 << 10) / ((int64_t)BULK_STAGES * 32 * row_bytes));
    warps = warps < 1 ? 1 : (warps > BULK_WARPS ? BULK_WARPS : warps);
    const size_t smem = (size_t)warps * BULK_STAGES * 32 * (size_t)row_bytes;
    // the shared-memory limit of a kernel is a per-device setting: remember what each device has been told
    static std::atomic<int> configured[64];
    int dev = 0;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= 64 || (int)smem > configured[dev].load(std::memory_order_relaxed)) {
        e = cudaFuncSetAttribute(k_gather_bulk, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        if (dev >= 0 && dev < 64) configured[dev].store((int)smem, std::memory_order_relaxed);
    }
    int per_sm = (int)((200u << 10) / (smem + 1024));
    per_sm = per_sm < 1 ? 1 : (per_sm > 16 ? 16 : per_sm);
    int64_t blocks = ((int64_t)count_bound + warps * 32 - 1) / (warps * 32);
    const int64_t cap = sm_count() * (int64_t)per_sm;
    blocks = limit_grid(blocks > cap ? cap : (blocks < 1 ? 1 : blocks));
    k_gather_bulk<<<(int)blocks, warps * 32, smem, s>>>((const char*)src, src_ld, (int)row_bytes, ids, d_count, count_bound,
                                                       (char*)dst, dst_ld, id_lo, id_hi);
    return cudaGetLastError();
}

cudaError_t gather_gave_up(cudaStream_t s, int* h_flag) {
    cudaError_t e = cudaMemcpyFromSymbolAsync(h_flag, g_gather_gave_up, sizeof(int), 0, cudaMemcpyDeviceToHost, s);
    if (e == cudaSuccess) e = cudaStreamSynchronize(s);
    return e;
}

template <typename V>
static void launch_t(const void* src, int64_t src_ld, int64_t row_bytes, const int32_t* ids, const int32_t* d_count,
                     int32_t count_bound, void* dst, int64_t dst_ld, int32_t blocks_per_sm, int id_lo, int id_hi,
                     cudaStream_t s) {
    const int units = (int)(row_bytes / (int64_t)sizeof(V));
    const int tpr = units < GT ? units : GT;
    const int rows_per_iter = GT / tpr;
    int64_t blocks = ((int64_t)count_bound + (int64_t)rows_per_iter * G_UNROLL - 1) / ((int64_t)rows_per_iter * G_UNROLL);
    // -1: the gather has the GPU to itself - a few long-lived blocks per SM; 0: a shape that also works beside others
    const int64_t cap = sm_count() * (int64_t)(blocks_per_sm > 0 ? blocks_per_sm : (blocks_per_sm < 0 ? 16 : GS_GATHER_GRID_PER_SM));
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
    // Default (and -1): the bulk-copy variant where it applies - measured on B200 with 2 M rows of 256 bytes, L2
    // flushed: 0.177 ms (5.9 TB/s) against 0.194 ms for the load/store kernel at its best grid; 2 to 4 warps per
    // block and 2 or 3 slices per warp are all within 2 % of each other, 4 slices or 8 warps are slower.
    // A positive blocks_per_sm asks for the load/store kernel with that grid.
    // It pays for rows of 128 to 512 bytes that start on 64-byte boundaries (measured, 2 M random rows, GB/s bulk vs
    // loads: 128 B 4664 / 4616, 192 B 4768 / 4565, 256 B 5858 / 5476, 320 B 5198 / 4897, 384 B 5916 / 5198); rows of
    // 64 bytes, or of 400 bytes on 16-byte boundaries, are faster with plain loads (2686 / 3348, 3917 / 4907).
    if (blocks_per_sm <= 0 && (all & 63) == 0 && row_bytes >= BULK_MIN_ROW && row_bytes <= BULK_MAX_ROW) {
        cudaError_t e = launch_bulk(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, (int)id_lo, (int)id_hi, s);
        count_launches(1);
        return e;
    }
    if ((all & 15) == 0) launch_t<uint4>(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, blocks_per_sm, (int)id_lo, (int)id_hi, s);
    else if ((all & 7) == 0) launch_t<uint2>(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, blocks_per_sm, (int)id_lo, (int)id_hi, s);
    else if ((all & 3) == 0) launch_t<uint32_t>(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, blocks_per_sm, (int)id_lo, (int)id_hi, s);
    else launch_t<uint16_t>(src, src_ld_bytes, row_bytes, ids, d_count, count_bound, dst, dst_ld_bytes, blocks_per_sm, (int)id_lo, (int)id_hi, s);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace gs
