// S3 alternatives to the direct-address table: where does an id first occur in "frontier ++ picked"?
//
//   hash  an open-addressing table sized to the batch - 1.5 x (n_k + m_k) entries of (id << 32 | position),
//         rebuilt at every sampling step: cleared, then every frontier id and every pick inserts itself
//         (compare-and-swap to claim a slot, atomicMin on the packed word where the id is already
//         there).  aux[e] keeps the slot of pick e, so the first-occurrence kernel needs one read.
//         The table follows the batch, not the graph: it stays in L2 where uint64[num_nodes] does not.
//   sort  a stable least-significant-digit radix sort (8-bit digits over the id's bits) of the words
//         (id << 32 | position); positions are the initial order, so inside a run of equal ids they
//         ascend and the head of the run is the first occurrence.  The head's position is handed to
//         every member of the run (tile-local max-scan of head indices + carry between tiles) and
//         scattered to aux[e].
//
// Both only produce what k_first_flags consumes; marking, scanning and k_relabel are shared with the
// direct method, so all three give identical blocks.  No kernel here waits for another block.
#include "gs_device.cuh"
#include "gs_internal.h"

namespace gs {

constexpr unsigned long long HASH_EMPTY = ~0ull;
constexpr int DD_THREADS = 256;

// 32-bit finalizer of MurmurHash3 (Appleby, public domain): spreads consecutive ids over the table.
__device__ __forceinline__ uint32_t mix32(uint32_t x) {
    x ^= x >> 16;
    x *= 0x85EBCA6Bu;
    x ^= x >> 13;
    x *= 0xC2B2AE35u;
    x ^= x >> 16;
    return x;
}

__global__ void __launch_bounds__(DD_THREADS) k_hash_clear(RelabelParams P) {
    chain_wait();
    if (__ldcg(P.hdr + HDR_STATUS) != 0) return;
    const long long keys = (long long)__ldcg(P.hdr + HDR_N + P.k) + __ldcg(P.hdr + HDR_M + P.k);
    long long cap = dedup_hash_capacity(keys);
    if (cap > P.scratch_entries) cap = P.scratch_entries;
    // two entries per store; the region starts 256-byte aligned and holds an even number of entries
    ulonglong2* t2 = reinterpret_cast<ulonglong2*>(P.scratch);
    const long long pairs = (cap + 1) / 2;
    for (long long i = (long long)blockIdx.x * DD_THREADS + threadIdx.x; i < pairs; i += (long long)gridDim.x * DD_THREADS)
        t2[i] = make_ulonglong2(HASH_EMPTY, HASH_EMPTY);
}

__global__ void __launch_bounds__(DD_THREADS) k_hash_insert(RelabelParams P) {
    chain_wait();
    int32_t* status = P.hdr + HDR_STATUS;
    if (__ldcg(status) != 0) return;
    const int n = __ldcg(P.hdr + HDR_N + P.k);
    const int m = __ldcg(P.hdr + HDR_M + P.k);
    const long long keys = (long long)n + m;
    const long long cap64 = dedup_hash_capacity(keys);
    if (cap64 > P.scratch_entries) {   // cannot happen with a workspace of the documented size
        if (blockIdx.x == 0 && threadIdx.x == 0) raise_status(status, GS_ERR_WORKSPACE);
        return;
    }
    const uint32_t cap = (uint32_t)cap64;
    for (long long i = (long long)blockIdx.x * DD_THREADS + threadIdx.x; i < keys; i += (long long)gridDim.x * DD_THREADS) {
        const uint32_t id = (uint32_t)(i < n ? P.frontier[i] : P.picked[i - n]);
        const unsigned long long mine = ((unsigned long long)id << 32) | (uint32_t)i;
        uint32_t slot = (uint32_t)(((unsigned long long)mix32(id) * cap) >> 32);
        // the load factor is at most 2/3, so a free or matching slot turns up after a few probes; the
        // probe count is bounded by the table size all the same
        // A plain read comes first: an id that is picked by thousands of rows would otherwise queue as many
        // atomics on one address; positions are inserted in roughly ascending order, so a later pick of the
        // same id nearly always finds a smaller position there already and has nothing to do.
        for (uint32_t probes = 0; probes < cap; ++probes) {
            unsigned long long cur = __ldcg(P.scratch + slot);
            if (cur == HASH_EMPTY) cur = atomicCAS(P.scratch + slot, HASH_EMPTY, mine);
            if (cur == HASH_EMPTY) break;                     // claimed
            if ((uint32_t)(cur >> 32) == id) {                // frontier ids are distinct, so one of the two is a pick
                if (cur > mine) atomicMin(P.scratch + slot, mine);
                break;
            }
            slot = slot + 1 == cap ? 0 : slot + 1;
        }
        if (i >= n) P.aux[i - n] = (int32_t)slot;
    }
}

cudaError_t launch_dedup_hash(const RelabelParams& p, int64_t n_bound, int64_t m_bound, cudaStream_t s) {
    const int64_t keys = n_bound + m_bound;
    int64_t blocks = (dedup_hash_capacity(keys) / 2 + DD_THREADS - 1) / DD_THREADS;
    if (blocks > sm_count() * 8) blocks = sm_count() * 8;
    launch_chained(k_hash_clear, limit_grid(blocks), DD_THREADS, s, p);
    blocks = (keys + DD_THREADS - 1) / DD_THREADS;
    if (blocks > sm_count() * 32) blocks = sm_count() * 32;
    launch_chained(k_hash_insert, limit_grid(blocks), DD_THREADS, s, p);
    count_launches(2);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- radix sort + unique
constexpr int SORT_TILE = 4096;                       // keys per block: 8 warps x 16 rounds x 32 lanes
constexpr int SORT_ROUNDS = SORT_TILE / DD_THREADS;   // 16

struct SortView {
    unsigned long long* a;      // key buffers
    unsigned long long* b;
    int32_t* hist;              // [256][tiles] digit counts, then exclusive offsets
    int32_t* tile_head;         // [tiles] last run head of each tile, then the carry into it
    int32_t* ticket;            // one counter, zeroed by the fill kernel
};

__host__ __device__ inline SortView sort_view(unsigned long long* scratch, long long keys_bound) {
    const long long tiles = (keys_bound + SORT_TILE - 1) / SORT_TILE + 1, tiles1k = (keys_bound + 1023) / 1024 + 1;
    SortView v;
    v.a = scratch;
    v.b = scratch + keys_bound + 32;
    int32_t* words = reinterpret_cast<int32_t*>(scratch + 2 * keys_bound + 64);
    v.hist = words;
    v.tile_head = words + 256 * tiles;
    v.ticket = v.tile_head + tiles1k;     // followed by the 256 digit totals
    return v;
}

struct SortParams {
    const int32_t* hdr;
    int32_t* status;
    int k;
    const int32_t* frontier;
    const int32_t* picked;
    int32_t* aux;
    SortView v;
    const unsigned long long* src;
    unsigned long long* dst;
    int shift;                   // bit position of the pass's digit inside the 64-bit word
    int tiles_bound;
};

__device__ __forceinline__ int sort_keys(const SortParams& P) {
    return __ldcg(P.hdr + HDR_N + P.k) + __ldcg(P.hdr + HDR_M + P.k);
}

__global__ void __launch_bounds__(DD_THREADS) k_sort_fill(SortParams P) {
    if (__ldcg(P.status) != 0) return;
    const int n = __ldcg(P.hdr + HDR_N + P.k);
    const int keys = sort_keys(P);
    if (blockIdx.x == 0 && threadIdx.x == 0) *P.v.ticket = 0;
    for (int i = blockIdx.x * DD_THREADS + threadIdx.x; i < keys; i += gridDim.x * DD_THREADS) {
        const uint32_t id = (uint32_t)(i < n ? P.frontier[i] : P.picked[i - n]);
        P.dst[i] = ((unsigned long long)id << 32) | (uint32_t)i;
    }
}

// Digit counts of one tile, per warp (a warp owns 512 consecutive keys of the tile, 32 per round).
// Lanes with the same digit are found with a warp match; the lowest of them adds the group's size.
__device__ __forceinline__ void tile_digit_counts(const SortParams& P, int tile, int keys, unsigned long long (&key)[SORT_ROUNDS],
                                                  int (*cnt)[256]) {
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int t = threadIdx.x; t < 8 * 256; t += DD_THREADS) (&cnt[0][0])[t] = 0;
    __syncthreads();
    const int wbase = tile * SORT_TILE + wid * (SORT_TILE / 8);
#pragma unroll
    for (int r = 0; r < SORT_ROUNDS; ++r) {
        const int i = wbase + r * 32 + lane;
        key[r] = i < keys ? __ldcg(P.src + i) : ~0ull;
        const uint32_t d = i < keys ? (uint32_t)(key[r] >> P.shift) & 255u : 256u;
        const uint32_t same = __match_any_sync(FULL, d);
        if (d < 256u && (same & lanemask_lt()) == 0) cnt[wid][d] += __popc(same);
        __syncwarp();
    }
    __syncthreads();
}

__global__ void __launch_bounds__(DD_THREADS) k_sort_hist(SortParams P) {
    __shared__ int cnt[8][256];
    if (__ldcg(P.status) != 0) return;
    const int keys = sort_keys(P);
    const int tiles = (keys + SORT_TILE - 1) / SORT_TILE;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        unsigned long long key[SORT_ROUNDS];
        tile_digit_counts(P, tile, keys, key, cnt);
        const int d = threadIdx.x;   // 256 threads = 256 digits
        int total = 0;
#pragma unroll
        for (int w = 0; w < 8; ++w) total += cnt[w][d];
        P.v.hist[(size_t)d * tiles + tile] = total;
        __syncthreads();
    }
}

// One block per digit: the digit's row sum ...
__global__ void __launch_bounds__(1024) k_sort_rowsum(SortParams P, int32_t* rowsum) {
    __shared__ int warp_sums[33];
    if (__ldcg(P.status) != 0) return;
    const int keys = sort_keys(P);
    const int tiles = (keys + SORT_TILE - 1) / SORT_TILE;
    const int d = blockIdx.x;
    int acc = 0;
    for (int t = threadIdx.x; t < tiles; t += 1024) acc += __ldcg(P.v.hist + (size_t)d * tiles + t);
    int total;
    block_exclusive_scan<1024>(acc, warp_sums, &total);
    if (threadIdx.x == 0) rowsum[d] = total;
}

// ... then the exclusive offsets of its tiles, after the sums of all smaller digits.
__global__ void __launch_bounds__(1024) k_sort_rowscan(SortParams P, const int32_t* rowsum) {
    __shared__ int warp_sums[33];
    __shared__ int s_base;
    if (__ldcg(P.status) != 0) return;
    const int keys = sort_keys(P);
    const int tiles = (keys + SORT_TILE - 1) / SORT_TILE;
    const int d = blockIdx.x;
    int mine = (threadIdx.x < 256 && (int)threadIdx.x < d) ? __ldcg(rowsum + threadIdx.x) : 0;
    int total;
    block_exclusive_scan<1024>(mine, warp_sums, &total);
    if (threadIdx.x == 0) s_base = total;
    __syncthreads();
    const int base = s_base;
    const int sum = scan_tiles_in_place<1024>(P.v.hist + (size_t)d * tiles, tiles, warp_sums);
    (void)sum;
    __syncthreads();
    for (int t = threadIdx.x; t < tiles; t += 1024) P.v.hist[(size_t)d * tiles + t] += base;
}

__global__ void __launch_bounds__(DD_THREADS) k_sort_scatter(SortParams P) {
    __shared__ int cnt[8][256];
    if (__ldcg(P.status) != 0) return;
    const int keys = sort_keys(P);
    const int tiles = (keys + SORT_TILE - 1) / SORT_TILE;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        unsigned long long key[SORT_ROUNDS];
        tile_digit_counts(P, tile, keys, key, cnt);
        {   // counts -> first output position of each (warp, digit)
            const int d = threadIdx.x;
            int run = __ldcg(P.v.hist + (size_t)d * tiles + tile);
#pragma unroll
            for (int w = 0; w < 8; ++w) {
                const int c = cnt[w][d];
                cnt[w][d] = run;
                run += c;
            }
        }
        __syncthreads();
        const int wbase = tile * SORT_TILE + wid * (SORT_TILE / 8);
#pragma unroll
        for (int r = 0; r < SORT_ROUNDS; ++r) {
            const int i = wbase + r * 32 + lane;
            const uint32_t d = i < keys ? (uint32_t)(key[r] >> P.shift) & 255u : 256u;
            const uint32_t same = __match_any_sync(FULL, d);
            int pos = 0;
            if (d < 256u) pos = cnt[wid][d] + __popc(same & lanemask_lt());
            __syncwarp();
            if (d < 256u && (same & lanemask_lt()) == 0) cnt[wid][d] += __popc(same);
            __syncwarp();
            if (d < 256u) P.dst[pos] = key[r];
        }
        __syncthreads();
    }
}

// Sorted keys in P.src.  Per tile: the largest index of a run head (-1 if none); the last block to
// finish turns these into the carry of each tile (the last head before the tile).
__global__ void __launch_bounds__(1024) k_sort_heads(SortParams P) {
    __shared__ int warp_max[32];
    __shared__ int is_last;
    if (__ldcg(P.status) != 0) return;
    const int keys = sort_keys(P);
    const int tiles = keys > 0 ? (keys + 1023) / 1024 : 1;
    if (threadIdx.x == 0) is_last = 0;
    __syncthreads();
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int i = tile * 1024 + threadIdx.x;
        int head = -1;
        if (i < keys) {
            const unsigned long long x = __ldcg(P.src + i);
            const bool is_head = i == 0 || (uint32_t)(__ldcg(P.src + i - 1) >> 32) != (uint32_t)(x >> 32);
            if (is_head) head = i;
        }
        const int wm = __reduce_max_sync(FULL, head);
        if ((threadIdx.x & 31) == 0) warp_max[threadIdx.x >> 5] = wm;
        __syncthreads();
        if (threadIdx.x < 32) {
            const int bm = __reduce_max_sync(FULL, warp_max[threadIdx.x]);
            if (threadIdx.x == 0) {
                P.v.tile_head[tile] = bm;
                __threadfence();
                is_last = (atomicAdd(P.v.ticket, 1) == tiles - 1);
            }
        }
        __syncthreads();
        if (is_last) break;
    }
    if (!is_last) return;
    __threadfence();
    // exclusive running maximum over the tiles, in place (one block; tiles are few)
    int carry = -1;
    for (int base = 0; base < tiles; base += 1024) {
        const int t = base + (int)threadIdx.x;
        const int x = t < tiles ? __ldcg(P.v.tile_head + t) : -1;
        int incl = x;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(FULL, incl, d);
            if ((int)(threadIdx.x & 31) >= d) incl = max(incl, y);
        }
        __syncthreads();
        if ((threadIdx.x & 31) == 31) warp_max[threadIdx.x >> 5] = incl;
        __syncthreads();
        int before = carry;
        for (int w = 0; w < (int)(threadIdx.x >> 5); ++w) before = max(before, warp_max[w]);
        const int up = __shfl_up_sync(FULL, incl, 1);
        const int excl = max(before, (threadIdx.x & 31) ? up : -1);
        if (t < tiles) P.v.tile_head[t] = excl;
        int all = carry;
        for (int w = 0; w < 32; ++w) all = max(all, warp_max[w]);
        carry = all;
        __syncthreads();
    }
}

// Every member of a run learns the position of the run's head; picks write it to aux.
__global__ void __launch_bounds__(1024) k_sort_resolve(SortParams P) {
    __shared__ int warp_max[32];
    if (__ldcg(P.status) != 0) return;
    const int n = __ldcg(P.hdr + HDR_N + P.k);
    const int keys = sort_keys(P);
    const int tiles = (keys + 1023) / 1024;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
        const int i = tile * 1024 + threadIdx.x;
        unsigned long long x = 0;
        int head = -1;
        if (i < keys) {
            x = __ldcg(P.src + i);
            if (i == 0 || (uint32_t)(__ldcg(P.src + i - 1) >> 32) != (uint32_t)(x >> 32)) head = i;
        }
        int incl = head;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(FULL, incl, d);
            if (lane >= d) incl = max(incl, y);
        }
        if (lane == 31) warp_max[wid] = incl;
        __syncthreads();
        int before = __ldcg(P.v.tile_head + tile);
        for (int w = 0; w < wid; ++w) before = max(before, warp_max[w]);
        const int leader = max(incl, before);
        if (i < keys && (uint32_t)x >= (uint32_t)n) {
            const uint32_t first = (uint32_t)__ldcg(P.src + leader);   // leader >= 0: index 0 is a head
            P.aux[(uint32_t)x - (uint32_t)n] = (int32_t)first;
        }
        __syncthreads();
    }
}

cudaError_t launch_dedup_sort(const RelabelParams& p, int64_t n_bound, int64_t m_bound, cudaStream_t s) {
    const int64_t keys = n_bound + m_bound;
    SortParams P{};
    P.hdr = p.hdr;
    P.status = p.hdr + HDR_STATUS;
    P.k = p.k;
    P.frontier = p.frontier;
    P.picked = p.picked;
    P.aux = p.aux;
    P.v = sort_view(p.scratch, keys);
    const int64_t tiles = (keys + SORT_TILE - 1) / SORT_TILE;
    int64_t grid = tiles < sm_count() * 8 ? tiles : sm_count() * 8;
    grid = limit_grid(grid < 1 ? 1 : grid);
    // the 256 row sums live behind the ticket word
    int32_t* rowsum = P.v.ticket + 4;
    P.dst = P.v.a;
    k_sort_fill<<<(int)grid, DD_THREADS, 0, s>>>(P);
    int launched = 1;
    unsigned long long* cur = P.v.a;
    unsigned long long* other = P.v.b;
    const int passes = (p.id_bits + 7) / 8;
    for (int pass = 0; pass < passes; ++pass) {
        P.src = cur;
        P.dst = other;
        P.shift = 32 + 8 * pass;
        k_sort_hist<<<(int)grid, DD_THREADS, 0, s>>>(P);
        k_sort_rowsum<<<256, 1024, 0, s>>>(P, rowsum);
        k_sort_rowscan<<<256, 1024, 0, s>>>(P, rowsum);
        k_sort_scatter<<<(int)grid, DD_THREADS, 0, s>>>(P);
        launched += 4;
        unsigned long long* t = cur;
        cur = other;
        other = t;
    }
    P.src = cur;
    int64_t tiles1k = (keys + 1023) / 1024;
    int64_t g2 = tiles1k < sm_count() * 2 ? tiles1k : sm_count() * 2;
    g2 = limit_grid(g2 < 1 ? 1 : g2);
    k_sort_heads<<<(int)g2, 1024, 0, s>>>(P);
    k_sort_resolve<<<(int)g2, 1024, 0, s>>>(P);
    count_launches(launched + 2);
    return cudaGetLastError();
}

}  // namespace gs
