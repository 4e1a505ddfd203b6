// Row counts + block CSR offsets (S4) and dedup / relabel (S3).
//
// Both are "tile-local scan, last block scans the tile sums" kernels: no block ever waits for
// another one, so there is no spin anywhere.
#include "gs_device.cuh"
#include "gs_internal.h"

namespace gs {

// ---------------------------------------------------------------- row counts
// Per frontier node p: count(p) = min(f, deg(frontier[p])) - the number of picks is known from the
// degree alone, so the block CSR offsets exist before anything is sampled.  Step 0 also copies
// the seeds into the frontier, validates them and preloads the relabel table with their positions.
__global__ void __launch_bounds__(1024) k_row_counts(CountParams P) {
    chain_wait();
    __shared__ int warp_sums[33];
    __shared__ int is_last;
    __shared__ int s_status;
    int32_t* status = P.hdr + HDR_STATUS;
    if (threadIdx.x == 0) {
        s_status = __ldcg(status);
        is_last = 0;
    }
    __syncthreads();
    if (s_status != 0) return;  // block-uniform: the barriers below stay convergent
    int n = (P.k == 0) ? P.n_host : __ldcg(P.hdr + HDR_N + P.k);
    if (P.k == 0 && P.d_n0) n = min(n, max(0, __ldcg(P.d_n0)));
    // a capped grid walks the tiles that hold frontier nodes (the host only knows an upper bound of n)
    const int tiles = (n + SCAN_A_TILE - 1) / SCAN_A_TILE;
    const int refresh_from = P.d_refresh_from ? __ldcg(P.d_refresh_from) : 0;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const int p = tile * SCAN_A_TILE + threadIdx.x;
    int c = 0;
    int nch = 0;   // scan work items of this node
    unsigned quads = 0, refreshed = 0;
    if (p < n) {
        int v;
        if (P.k == 0) {
            v = P.seeds[p];
            if (v < 0 || (int64_t)v >= P.g.num_nodes) {
                raise_status(status, GS_ERR_RANGE);
                v = -1;
            } else {
                P.frontier[p] = v;
                if (!P.no_stamp) {
                    const unsigned long long mine = ((unsigned long long)P.stamp << 32) | (unsigned)p;
                    const unsigned long long old = atomicMin(P.table + v, mine);
                    if ((uint32_t)(old >> 32) == P.stamp) raise_status(status, GS_ERR_DUP_SEED);
                }
            }
        } else {
            v = P.frontier[p];
        }
        if (v >= 0 && P.reply) {
            // sharded run, requester side: the owners have sampled; a row's picks are the non-negative prefix
            const int sl = P.slot ? P.slot[p] : p;
            if ((unsigned)sl >= (unsigned)(P.reply_rows > 0 ? P.reply_rows : n)) {
                raise_status(status, GS_ERR_RANGE);   // not a row of the reply: the node gets no picks
            } else {
                const int32_t* row = P.reply + (int64_t)sl * P.f;
                while (c < P.f && __ldg(row + c) >= 0) ++c;
            }
        } else if (v >= 0) {
            const int64_t deg = P.g.indptr[v + 1] - P.g.indptr[v];
            c = deg < (int64_t)P.f ? (int)deg : P.f;
            if (P.r > 0 && deg > (int64_t)SMALL_DEGREE && deg > (int64_t)P.W && p >= refresh_from) {
                const int64_t nq = (deg + 3) >> 2;
                nch = (int)((nq + HUB_CHUNK_QUADS - 1) / HUB_CHUNK_QUADS);
                quads = (unsigned)nq;
            }
            if (P.r > 0 && deg > (int64_t)P.W && p >= refresh_from) refreshed = 1;
        }
    }
    int total;
    const int excl = block_exclusive_scan<SCAN_A_TILE>(c, warp_sums, &total);
    if (p < n) P.blk_indptr[p] = excl;
    int total2 = 0;
    {
        const unsigned wq = __reduce_add_sync(FULL, quads), wr = __reduce_add_sync(FULL, refreshed);
        if ((threadIdx.x & 31) == 0 && wr) {
            atomicAdd((unsigned*)(P.hdr + HDR_STAT_QUADS), wq);
            atomicAdd((unsigned*)(P.hdr + HDR_STAT_REFRESHED), wr);
        }
        const int excl2 = block_exclusive_scan<SCAN_A_TILE>(nch, warp_sums, &total2);
        if (p < n) P.item_start[p] = excl2;
    }
    if (threadIdx.x == 0) {
        P.tile_sums2[tile] = total2;
        P.tile_sums[tile] = total;
        __threadfence();
        const int ticket = atomicAdd(P.hdr + HDR_TICKET_A + P.k, 1);
        is_last = (ticket == tiles - 1);
    }
    __syncthreads();
    if (is_last) break;   // every tile is done (this block's later ones included): finish below
    }
    if (!is_last) return;
    __threadfence();
    const int m = scan_tiles_in_place<SCAN_A_TILE>(P.tile_sums, tiles, warp_sums);
    const int items = scan_tiles_in_place<SCAN_A_TILE>(P.tile_sums2, tiles, warp_sums);
    if (threadIdx.x == 0) {
        P.hdr[HDR_M + P.k] = m;
        P.hdr[HDR_ITEMS + P.k] = items;
        if (P.k == 0) P.hdr[HDR_N] = n;
    }
}

__global__ void __launch_bounds__(1024) k_row_offsets(CountParams P) {
    chain_wait();
    if (__ldcg(P.hdr + HDR_STATUS) != 0) return;
    int n = (P.k == 0) ? P.n_host : __ldcg(P.hdr + HDR_N + P.k);
    if (P.k == 0 && P.d_n0) n = min(n, max(0, __ldcg(P.d_n0)));
    for (int t = blockIdx.x; t <= n / SCAN_A_TILE; t += gridDim.x) {   // the tile of position n takes part too
    const int p = t * SCAN_A_TILE + threadIdx.x;
    if (p < n) P.blk_indptr[p] += P.tile_sums[p / SCAN_A_TILE];
    else if (p == n) P.blk_indptr[n] = __ldcg(P.hdr + HDR_M + P.k);
    // scan work items: node p owns items [item_start[p], item_start[p+1]), one per chunk of its row
    int first = 0, next = 0;
    if (p < n) {
        const int tile = p / SCAN_A_TILE;
        first = P.item_start[p] + P.tile_sums2[tile];
        if (p + 1 >= n) next = __ldcg(P.hdr + HDR_ITEMS + P.k);
        else if ((p + 1) % SCAN_A_TILE == 0) next = P.tile_sums2[tile + 1];   // first node of the next tile
        else next = P.item_start[p + 1] + P.tile_sums2[tile];
    }
    __syncthreads();   // tile-local values are all read before any is overwritten below
    // one descriptor per chunk of the node's row: the scan needs nothing else to start on it.  A thread writes the
    // few chunks of an ordinary row itself; the hundreds of a hub are written by its whole warp.
    int v = 0, deg = 0;
    if ((int64_t)next > P.scan_item_cap) next = (int)P.scan_item_cap;
    if (p < n) {
        P.item_start[p] = first;
        P.cand_count[p] = 0;
        if (first < next) {
            v = P.frontier[p];
            deg = (int)(P.g.indptr[v + 1] - P.g.indptr[v]);
            if (next - first <= 4)
                for (int w = first; w < next; ++w) P.items[w] = make_int4(p, v, deg, w - first);
        }
    } else if (p == n) {
        P.item_start[n] = __ldcg(P.hdr + HDR_ITEMS + P.k);
    }
    unsigned wide = __ballot_sync(FULL, next - first > 4);
    while (wide) {
        const int src = __ffs(wide) - 1;
        wide &= wide - 1;
        const int hp = __shfl_sync(FULL, p, src), hv = __shfl_sync(FULL, v, src), hd = __shfl_sync(FULL, deg, src);
        const int hf = __shfl_sync(FULL, first, src), hn = __shfl_sync(FULL, next, src);
        for (int w = hf + (int)(threadIdx.x & 31); w < hn; w += 32) P.items[w] = make_int4(hp, hv, hd, w - hf);
    }
    }
}

cudaError_t launch_row_counts(const CountParams& p, int64_t n_bound, cudaStream_t s) {
    // at most two resident blocks of 1,024 threads per SM; blocks walk the tiles that exist
    int64_t tiles = n_bound / SCAN_A_TILE + 1;
    if (tiles > sm_count() * 2) tiles = sm_count() * 2;
    tiles = limit_grid(tiles);
    launch_chained(k_row_counts, tiles, SCAN_A_TILE, s, p);
    launch_chained(k_row_offsets, tiles, SCAN_A_TILE, s, p);
    count_launches(2);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- dedup + relabel
// The picks were written with atomicMin(table[id], position) where the position of pick e in the
// list "frontier ++ picked" is n + e; frontier members already sit in the table with positions
// < n.  Pass 1 marks each id's first occurrence and scans the marks; pass 2 turns them into
// block-local ids, appends the new ids to the frontier and stores their final position in the
// table (which is exactly the preload the next step needs).
//
// aux[e] holds, for a first occurrence, -(tile-local rank)-1, otherwise the table position.
constexpr int FF_THREADS = 256;                 // 8 warps, each owns 512 consecutive picks of the tile
static_assert(SCAN_E_TILE == FF_THREADS * 16, "tile = 16 picks per thread");

// METHOD says where the first position of a pick's id comes from: the direct-address table (read with the
// id), the batch-sized hash table (aux[e] holds the id's slot), or aux[e] itself (the sort left it there).
template <int METHOD>
__global__ void __launch_bounds__(FF_THREADS) k_first_flags(RelabelParams P) {
    chain_wait();
    __shared__ int warp_sums[33];
    __shared__ int s_wtot[FF_THREADS / 32];
    __shared__ int is_last;
    __shared__ int s_status;
    if (threadIdx.x == 0) {
        s_status = __ldcg(P.hdr + HDR_STATUS);
        is_last = 0;
    }
    __syncthreads();
    if (s_status != 0) return;  // block-uniform
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int n = __ldcg(P.hdr + HDR_N + P.k);
    const int m = __ldcg(P.hdr + HDR_M + P.k);
    // a capped grid walks the tiles that hold picks (at least one, to publish n_{k+1})
    const int tiles = m > 0 ? (m + SCAN_E_TILE - 1) / SCAN_E_TILE : 1;
    for (int tile = blockIdx.x; tile < tiles; tile += gridDim.x) {
    const int wbase = tile * SCAN_E_TILE + wid * 512;
    // 16 independent table probes per thread are in flight before anything is consumed
    int id[4][4];
    int pos[4][4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int e0 = wbase + j * 128 + lane * 4;
        int4 v = make_int4(0, 0, 0, 0);
        if (e0 < m) v = *reinterpret_cast<const int4*>((METHOD == DEDUP_DIRECT ? P.picked : P.aux) + e0);  // buffers are padded to 4
        id[j][0] = v.x; id[j][1] = v.y; id[j][2] = v.z; id[j][3] = v.w;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int e0 = wbase + j * 128 + lane * 4;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            if (METHOD == DEDUP_DIRECT) pos[j][i] = (e0 + i < m) ? (int)(uint32_t)__ldcg(P.table + id[j][i]) : -1;
            else if (METHOD == DEDUP_HASH) pos[j][i] = (e0 + i < m) ? (int)(uint32_t)__ldcg(P.scratch + id[j][i]) : -1;
            else pos[j][i] = (e0 + i < m) ? id[j][i] : -1;
        }
    }
    int cnt[4], incl[4], before[4];
    int wtotal = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int e0 = wbase + j * 128 + lane * 4;
        int c = 0;
#pragma unroll
        for (int i = 0; i < 4; ++i) c += (e0 + i < m && pos[j][i] == n + e0 + i) ? 1 : 0;
        cnt[j] = c;
        int x = c;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            const int y = __shfl_up_sync(FULL, x, d);
            if (lane >= d) x += y;
        }
        incl[j] = x;
        before[j] = wtotal;
        wtotal += __shfl_sync(FULL, x, 31);
    }
    if (lane == 0) s_wtot[wid] = wtotal;
    __syncthreads();
    int woff = 0, total = 0;
#pragma unroll
    for (int w = 0; w < FF_THREADS / 32; ++w) {
        const int t = s_wtot[w];
        if (w < wid) woff += t;
        total += t;
    }
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const int e0 = wbase + j * 128 + lane * 4;
        if (e0 < m) {
            int run = woff + before[j] + incl[j] - cnt[j];
            int out[4];
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const bool first = (e0 + i < m) && pos[j][i] == n + e0 + i;
                out[i] = first ? -run - 1 : pos[j][i];
                run += first ? 1 : 0;
            }
            *reinterpret_cast<int4*>(P.aux + e0) = make_int4(out[0], out[1], out[2], out[3]);
        }
    }
    if (threadIdx.x == 0) {
        P.tile_sums[tile] = total;
        __threadfence();
        const int ticket = atomicAdd(P.hdr + HDR_TICKET_E + P.k, 1);
        is_last = (ticket == tiles - 1);
    }
    __syncthreads();   // also keeps s_wtot of this tile intact until every warp has read it
    if (is_last) break;
    }
    if (!is_last) return;
    __threadfence();
    const int fresh = scan_tiles_in_place<FF_THREADS>(P.tile_sums, tiles, warp_sums);
    if (threadIdx.x == 0) P.hdr[HDR_N + P.k + 1] = n + fresh;
}

// Eight consecutive picks per thread, so that the dependent probes of eight items overlap.
constexpr int RL_PICKS = 8;

__global__ void __launch_bounds__(256) k_relabel(RelabelParams P) {
    chain_wait();
    if (__ldcg(P.hdr + HDR_STATUS) != 0) return;
    const int n = __ldcg(P.hdr + HDR_N + P.k);
    const int m = __ldcg(P.hdr + HDR_M + P.k);
    for (int e0 = RL_PICKS * (blockIdx.x * blockDim.x + threadIdx.x); e0 < m; e0 += RL_PICKS * gridDim.x * blockDim.x) {
        int val[RL_PICKS];
#pragma unroll
        for (int q = 0; q < RL_PICKS / 4; ++q) {
            int4 a = make_int4(0, 0, 0, 0);
            if (e0 + 4 * q < m) a = *reinterpret_cast<const int4*>(P.aux + e0 + 4 * q);   // padded to 4
            val[4 * q] = a.x; val[4 * q + 1] = a.y; val[4 * q + 2] = a.z; val[4 * q + 3] = a.w;
        }
        int ref[RL_PICKS], tile[RL_PICKS], id[RL_PICKS];
#pragma unroll
        for (int i = 0; i < RL_PICKS; ++i) {
            // first occurrence: own mark; later occurrence of a new id: the mark of its first occurrence
            const int src = (val[i] < 0) ? e0 + i : (val[i] >= n ? val[i] - n : -1);
            ref[i] = val[i];
            tile[i] = 0;
            id[i] = 0;
            if (e0 + i < m && src >= 0) {
                if (val[i] >= 0) ref[i] = P.aux[src];
                else id[i] = P.picked[e0 + i];
                tile[i] = P.tile_sums[src / SCAN_E_TILE];
            }
        }
        int out[RL_PICKS];
#pragma unroll
        for (int i = 0; i < RL_PICKS; ++i) {
            int loc = val[i];
            if (e0 + i < m && (val[i] < 0 || val[i] >= n)) {
                loc = n + (-ref[i] - 1) + tile[i];
                if (val[i] < 0 && (int64_t)loc < P.n_cap) {
                    P.frontier[loc] = id[i];
                    if (P.table) P.table[id[i]] = ((unsigned long long)P.stamp << 32) | (unsigned)loc;
                }
            }
            out[i] = loc;
        }
#pragma unroll
        for (int q = 0; q < RL_PICKS / 4; ++q) {
            const int e = e0 + 4 * q;
            if (e + 3 < m) {
                *reinterpret_cast<int4*>(P.local + e) = make_int4(out[4 * q], out[4 * q + 1], out[4 * q + 2], out[4 * q + 3]);
            } else {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (e + i < m) P.local[e + i] = out[4 * q + i];
            }
        }
    }
}

cudaError_t launch_relabel(const RelabelParams& p, int64_t n_bound, int64_t m_bound, cudaStream_t s) {
    if (m_bound <= 0) m_bound = 1;
    if (p.method == DEDUP_HASH) {
        cudaError_t e = launch_dedup_hash(p, n_bound, m_bound, s);
        if (e != cudaSuccess) return e;
    } else if (p.method == DEDUP_SORT) {
        cudaError_t e = launch_dedup_sort(p, n_bound, m_bound, s);
        if (e != cudaSuccess) return e;
    }
    int64_t tiles = (m_bound + SCAN_E_TILE - 1) / SCAN_E_TILE;
    if (tiles > sm_count() * 16) tiles = sm_count() * 16;    // blocks walk the tiles; enough of them that a usual batch has one tile each
    tiles = limit_grid(tiles);
    if (p.method == DEDUP_HASH) launch_chained(k_first_flags<DEDUP_HASH>, tiles, FF_THREADS, s, p);
    else if (p.method == DEDUP_SORT) launch_chained(k_first_flags<DEDUP_SORT>, tiles, FF_THREADS, s, p);
    else launch_chained(k_first_flags<DEDUP_DIRECT>, tiles, FF_THREADS, s, p);
    int64_t blocks = (m_bound + 256 * RL_PICKS - 1) / (256 * RL_PICKS);
    if (blocks > sm_count() * 16) blocks = sm_count() * 16;
    blocks = limit_grid(blocks);
    RelabelParams q = p;
    if (p.method != DEDUP_DIRECT) q.table = nullptr;
    launch_chained(k_relabel, blocks, 256, s, q);
    count_launches(2);
    return cudaGetLastError();
}

// ---------------------------------------------------------------- graph contract check
// One warp per row: offsets non-decreasing, the row inside [0, num_edges], neighbour ids inside
// [0, num_nodes) and strictly ascending (sorted, no duplicate).  The lowest offending row wins.
__device__ unsigned long long g_first_bad_row;

__global__ void __launch_bounds__(256) k_validate_graph(GraphView g, long long num_edges, unsigned long long* bad) {
    const int lane = threadIdx.x & 31;
    const long long warps = (long long)gridDim.x * (blockDim.x >> 5);
    for (long long v = (long long)blockIdx.x * (blockDim.x >> 5) + (threadIdx.x >> 5); v < g.num_nodes; v += warps) {
        const long long lo = g.indptr[v], hi = g.indptr[v + 1];
        bool wrong = lo > hi || lo < 0 || hi > num_edges || (v == 0 && lo != 0) || (v == g.num_nodes - 1 && hi != num_edges);
        if (!wrong)
            for (long long e = lo + lane; e < hi; e += 32) {
                const int32_t u = g.indices[e];
                if (u < 0 || (long long)u >= g.num_nodes || (e > lo && g.indices[e - 1] >= u)) wrong = true;
            }
        if (__any_sync(FULL, wrong) && lane == 0) atomicMin(bad, (unsigned long long)v);
    }
}

cudaError_t launch_validate_graph(const GraphView& g, int64_t num_edges, int64_t* h_first_bad_row, cudaStream_t s) {
    unsigned long long* d_bad = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&d_bad, g_first_bad_row);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(d_bad, 0xFF, sizeof(unsigned long long), s);
    if (e != cudaSuccess) return e;
    int64_t blocks = (g.num_nodes + 7) / 8;
    if (blocks > sm_count() * 16) blocks = sm_count() * 16;
    k_validate_graph<<<(int)blocks, 256, 0, s>>>(g, (long long)num_edges, d_bad);
    count_launches(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    unsigned long long h = 0;
    e = cudaMemcpyAsync(&h, d_bad, sizeof(h), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return e;
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return e;
    *h_first_bad_row = (h == ~0ull) ? -1 : (int64_t)h;
    return cudaSuccess;
}

// ---------------------------------------------------------------- dense part of a split cache
// Number of nodes with degree > theta (what gs_cache_bytes_split and gs_cache_init_split are sized from).
__device__ unsigned long long g_dense_count;

__global__ void __launch_bounds__(256) k_count_dense(GraphView g, long long theta, unsigned long long* out) {
    unsigned mine = 0;
    for (long long v = (long long)blockIdx.x * blockDim.x + threadIdx.x; v < g.num_nodes; v += (long long)gridDim.x * blockDim.x)
        mine += (g.indptr[v + 1] - g.indptr[v] > theta) ? 1u : 0u;
    mine = __reduce_add_sync(FULL, mine);
    if ((threadIdx.x & 31) == 0 && mine) atomicAdd(out, (unsigned long long)mine);
}

cudaError_t launch_count_dense(const GraphView& g, int32_t theta, int64_t* h_count, cudaStream_t s) {
    unsigned long long* d = nullptr;
    cudaError_t e = cudaGetSymbolAddress((void**)&d, g_dense_count);
    if (e != cudaSuccess) return e;
    e = cudaMemsetAsync(d, 0, sizeof(unsigned long long), s);
    if (e != cudaSuccess) return e;
    int64_t blocks = (g.num_nodes + 255) / 256;
    if (blocks > sm_count() * 16) blocks = sm_count() * 16;
    k_count_dense<<<(int)blocks, 256, 0, s>>>(g, (long long)theta, d);
    count_launches(1);
    e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    unsigned long long h = 0;
    e = cudaMemcpyAsync(&h, d, sizeof(h), cudaMemcpyDeviceToHost, s);
    if (e != cudaSuccess) return e;
    e = cudaStreamSynchronize(s);
    if (e != cudaSuccess) return e;
    *h_count = (int64_t)h;
    return cudaSuccess;
}

// ---------------------------------------------------------------- logical cache rows (parity / debug)
__global__ void k_read_rows(const int32_t* slots, const int32_t* row_index, int pitch, int W, const int32_t* nodes,
                            int n, int32_t* out) {
    const int i = blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n * W) return;
    const int row = i / W, j = i - row * W;
    const int64_t r = row_index ? (int64_t)row_index[nodes[row]] : (int64_t)nodes[row];
    out[i] = r >= 0 ? slots[r * pitch + j] : -1;   // nodes of the sparse part have no cache row
}

// Split cache: row_index[v] = rank of v among the nodes with degree > theta, -1 for the others.
// Same pattern as the other scans: tile-local scan, the last block scans the tile sums; a second
// kernel adds the tile offsets.
__global__ void __launch_bounds__(1024) k_row_index_local(GraphView g, int theta, int32_t* row_index,
                                                          int32_t* tile_sums, int32_t* ticket_and_total) {
    __shared__ int warp_sums[33];
    __shared__ int is_last;
    const int64_t v = (int64_t)blockIdx.x * 1024 + threadIdx.x;
    int dense = 0;
    if (v < g.num_nodes) dense = (g.indptr[v + 1] - g.indptr[v] > (int64_t)theta) ? 1 : 0;
    int total;
    const int excl = block_exclusive_scan<1024>(dense, warp_sums, &total);
    if (v < g.num_nodes) row_index[v] = dense ? excl : -1;
    if (threadIdx.x == 0) {
        tile_sums[blockIdx.x] = total;
        __threadfence();
        is_last = (atomicAdd(ticket_and_total, 1) == (int)gridDim.x - 1);
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    const int rows = scan_tiles_in_place<1024>(tile_sums, (int)gridDim.x, warp_sums);
    if (threadIdx.x == 0) ticket_and_total[1] = rows;
}

__global__ void __launch_bounds__(1024) k_row_index_offsets(int64_t num_nodes, int32_t* row_index, const int32_t* tile_sums) {
    const int64_t v = (int64_t)blockIdx.x * 1024 + threadIdx.x;
    if (v < num_nodes && row_index[v] >= 0) row_index[v] += tile_sums[blockIdx.x];
}

// d_dense_rows: two zeroed ints (ticket, result).
cudaError_t launch_build_row_index(const GraphView& g, int32_t theta, int32_t* row_index, int32_t* tile_sums,
                                   int32_t* d_dense_rows, cudaStream_t s) {
    const int tiles = (int)((g.num_nodes + 1023) / 1024);
    k_row_index_local<<<tiles, 1024, 0, s>>>(g, theta, row_index, tile_sums, d_dense_rows);
    k_row_index_offsets<<<tiles, 1024, 0, s>>>(g.num_nodes, row_index, tile_sums);
    count_launches(2);
    return cudaGetLastError();
}

cudaError_t launch_read_rows(const int32_t* slots, const int32_t* row_index, int32_t pitch, int32_t W,
                             const int32_t* nodes, int32_t n, int32_t* out, cudaStream_t s) {
    if (n <= 0) return cudaSuccess;
    const int64_t total = (int64_t)n * W;
    k_read_rows<<<(int)((total + 255) / 256), 256, 0, s>>>(slots, row_index, pitch, W, nodes, n, out);
    count_launches(1);
    return cudaGetLastError();
}

}  // namespace gs
