// S0 static pre-sample, S1 refresh (FCR / OTF, and the FBL / OTF Fetch variants) and S2 pick.
//
// Every selection is "the k items first in (key, index) order" with Philox keys that depend on
// (node, item index, step) only - not on the neighbour ids.  The scan over a node's deg edge
// offsets therefore reads no CSR bytes: it evaluates one Philox block per four offsets, keeps the
// offsets whose key is at or below a threshold chosen so that about lambda of them survive, and
// only then reads the few neighbour ids it needs.  If the survivors turn out not to be enough (or
// too many for the buffer) the node is redone with a larger lambda and finally with an exact
// running top-W, so the result never depends on the threshold.  The kernel is bound by integer
// ALU throughput (Philox), not by memory.
//
// Refill rule used (it follows from the refresh definition): the r refill winners are the first r
// entries, after removing retained neighbours, of the top-W list of ALL edge offsets in FILL
// order, because at most W - r retained neighbours can precede the r-th winner.
//
// Kernels:
//   k_scan + k_finish   every batch (see "split path" below): a pure Philox threshold scan over the
//                       rows above SMALL_DEGREE, then one warp per frontier node for eviction,
//                       refill, row update and pick.
//   k_refresh_pick      refresh (+ optional pick) fused in one warp per node, software-pipelined:
//                       while the neighbour ids of node i are in flight the warp already scans node
//                       i+1.  Used where every node of a range is refreshed - the static pre-sample
//                       and the whole-cache refresh.  Nodes above the hub degree are only
//                       registered, as a list of 4096-offset chunks.
//   k_refresh_pick_hub  one warp per chunk of a registered hub; candidates go to a per-hub buffer
//                       in global memory, and the warp that finishes a hub's last chunk completes
//                       the node.  Also redoes the long rows k_finish could not decide from their
//                       candidate lists.  No warp ever waits for another one.
#include "gs_device.cuh"
#include "gs_internal.h"

namespace gs {

#ifndef GS_SCAN_BATCH_DIV
#define GS_SCAN_BATCH_DIV 16
#endif
#ifndef GS_SCAN_MIN_BLOCKS
#define GS_SCAN_MIN_BLOCKS 3
#endif
#ifndef GS_FINISH_MIN_BLOCKS
#define GS_FINISH_MIN_BLOCKS 4
#endif
constexpr int RP_THREADS = 256;
constexpr int RP_WARPS = RP_THREADS / 32;
constexpr int RETRY_QUEUE_DEGREE = 2048;  // split path: longer rows that need a rescan go to the hub kernel
static_assert(CAND_CAP == HUB_CAND_CAP, "hub buffers are copied into a warp buffer");

// First slot of node v's cache row; negative for a node of the sparse part of a split cache.
__device__ __forceinline__ int64_t row_offset(const StepParams& P, int32_t v) {
    const int64_t r = P.row_index ? (int64_t)__ldg(P.row_index + v) : (int64_t)v;
    return r * P.pitch;
}

__device__ __forceinline__ uint32_t threshold_for(float lambda, uint32_t deg) {
    // inclusive key threshold: about lambda of deg uniform 32-bit keys fall at or below it
    if (deg <= (uint32_t)CAND_CAP) return 0xFFFFFFFFu;
    const float t = lambda / (float)deg * 4294967296.0f;
    return t >= 4294967040.0f ? 0xFFFFFFFFu : (uint32_t)t;
}

// One warp scans quads [q_begin, q_end) of the node's offsets (quad q = offsets 4q..4q+3) and
// appends (key << 32 | offset) of every offset with key <= tinc to buf.  `count` is the warp's
// running count (entries beyond CAND_CAP are counted but not stored).
__device__ __forceinline__ int warp_collect(const StepParams& P, int32_t v, uint32_t deg, uint32_t q_begin,
                                            uint32_t q_end, uint32_t tinc, unsigned long long* buf, int count,
                                            int lane) {
    const uint32_t lt = lanemask_lt();
    // consecutive quads of one row: the row form of the key function (see philox_row_block)
    const RowKeys rkeys = philox_row_keys((uint32_t)v, P.step, P.word_fill, P.rk);
    unsigned long long p0 = (unsigned long long)PHILOX_M0 * (unsigned long long)(q_begin + (uint32_t)lane);
    for (uint32_t qb = q_begin; qb < q_end; qb += 32, p0 = add64(p0, 32ull * PHILOX_M0)) {
        const uint32_t q = qb + lane;
        const uint4 o = philox_row_block(p0, rkeys, P.rk);
        const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
        const bool inq = q < q_end;
        const bool any = inq && (__vimin3_u32(min(kk[0], kk[1]), kk[2], kk[3]) <= tinc);
        if (__ballot_sync(FULL, any) == 0) continue;   // the common case: nothing below the threshold
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const uint32_t off = 4u * q + w;
            const bool hit = inq && (off < deg) && (kk[w] <= tinc);
            const uint32_t b = __ballot_sync(FULL, hit);
            if (b) {
                if (hit) {
                    const int pos = count + __popc(b & lt);
                    if (pos < CAND_CAP) buf[pos] = ((unsigned long long)kk[w] << 32) | off;
                }
                count += __popc(b);
            }
        }
    }
    __syncwarp();
    return count;
}

// Exact fallback: one warp keeps the W smallest (key, offset) pairs in a sorted list, one per
// lane, while scanning every offset.  Leaves them in buf[0..W) in order.
__device__ __noinline__ void warp_exact_top(const StepParams& P, int32_t v, uint32_t deg, unsigned long long* buf,
                                            int lane) {
    const int W = P.W;
    unsigned long long cur = ~0ull;
    const uint32_t nq = (deg + 3u) >> 2;
    for (uint32_t qb = 0; qb < nq; qb += 32) {
        const uint32_t q = qb + lane;
        const uint4 o = philox4x32_10_rk(q, (uint32_t)v, P.step, P.word_fill, P.rk);
        const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const uint32_t off = 4u * q + w;
            const unsigned long long val =
                (q < nq && off < deg) ? (((unsigned long long)kk[w] << 32) | off) : ~0ull;
            unsigned long long thr = __shfl_sync(FULL, cur, W - 1);
            uint32_t b = __ballot_sync(FULL, val < thr);
            while (b) {
                const int src = __ffs(b) - 1;
                b &= b - 1;
                const unsigned long long x = __shfl_sync(FULL, val, src);
                if (x < thr) {
                    const int pos = __popc(__ballot_sync(FULL, cur < x));
                    const unsigned long long up = __shfl_up_sync(FULL, cur, 1);
                    if (lane > pos) cur = up;
                    else if (lane == pos) cur = x;
                    if (lane >= W) cur = ~0ull;
                    thr = __shfl_sync(FULL, cur, W - 1);
                }
            }
        }
    }
    if (lane < W) buf[lane] = cur;
    __syncwarp();
}

// Removes and returns the smallest of the candidates a warp holds four-per-lane.
__device__ __forceinline__ unsigned long long warp_pop_min(unsigned long long (&it)[4]) {
    unsigned long long loc = it[0];
#pragma unroll
    for (int j = 1; j < 4; ++j) loc = it[j] < loc ? it[j] : loc;
    const uint32_t hi = (uint32_t)(loc >> 32);
    const uint32_t mhi = __reduce_min_sync(FULL, hi);
    const uint32_t lo = (hi == mhi) ? (uint32_t)loc : 0xFFFFFFFFu;
    const uint32_t mlo = __reduce_min_sync(FULL, lo);
    const unsigned long long best = ((unsigned long long)mhi << 32) | mlo;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (it[j] == best) it[j] = ~0ull;  // offsets are distinct, so exactly one copy exists
    return best;
}

// Refill of one node, split in two so that the neighbour-id loads issued by begin() can be in
// flight while the warp works on something else.
struct Refill {
    unsigned long long it[4];  // candidates, four per lane
    int c;                     // candidate count, -1 = unusable (too few / overflow)
    int taken, g;              // extracted so far; size of the batch whose ids are in flight
    bool whole;                // candidates are all offsets, or the exact top-W
    uint32_t my_off;           // lane t holds the t-th candidate in FILL order ...
    int32_t my_nb;             // ... and its neighbour id

    __device__ __forceinline__ void extract(const StepParams& P, int64_t row_start, int lane) {
        for (int t = 0; t < g; ++t) {
            const unsigned long long best = warp_pop_min(it);
            if (lane == taken + t) my_off = (uint32_t)best;
        }
        if (lane >= taken && lane < taken + g) my_nb = __ldg(P.g.indices + row_start + my_off);
    }

    __device__ __forceinline__ void begin(const StepParams& P, int64_t row_start, const unsigned long long* buf,
                                          int count, bool all, int r, int lane) {
        c = count;
        whole = all;
        taken = 0;
        g = 0;
        my_off = 0;
        my_nb = -1;
        if (count > CAND_CAP || count < r) { c = -1; return; }
#pragma unroll
        for (int j = 0; j < 4; ++j) it[j] = (lane + 32 * j < c) ? buf[lane + 32 * j] : ~0ull;
        const int limit = c < P.W ? c : P.W;
        g = r < limit ? r : limit;
        extract(P, row_start, lane);
    }

    // Completes the refill into `slot`.  Returns false if the candidates cannot decide it.
    __device__ __forceinline__ bool finish(const StepParams& P, int64_t row_start, uint32_t evict_mask,
                                           int32_t& slot, int lane) {
        if (c < 0) return false;
        const int W = P.W;
        const int r = __popc(evict_mask);
        const int limit = c < W ? c : W;  // never more than the top-W matter
        const bool retained = (lane < W) && !((evict_mask >> lane) & 1u);
        uint32_t valid = 0;
        while (true) {
            for (int t = taken; t < taken + g; ++t) {
                const int32_t x = __shfl_sync(FULL, my_nb, t);
                const uint32_t hit = __ballot_sync(FULL, retained && slot == x);
                if (hit == 0) valid |= 1u << t;
            }
            taken += g;
            if (__popc(valid) >= r) break;
            if (taken >= limit) {
                if (whole || c >= W) break;  // the whole top-W was examined (cannot lack winners)
                return false;
            }
            g = r - __popc(valid);
            if (g > limit - taken) g = limit - taken;
            extract(P, row_start, lane);
        }
        if (__popc(valid) < r) return false;
        // t-th valid candidate -> t-th evicted slot (ascending slot index)
        const bool ev = (evict_mask >> lane) & 1u;
        const int e = __popc(evict_mask & lanemask_lt());
        const int src = ev ? (int)__fns(valid, 0, e + 1) : 0;
        const int32_t nv = __shfl_sync(FULL, my_nb, src & 31);
        if (ev) slot = nv;
        return true;
    }
};

// Removes and returns the largest of the candidates a warp holds four-per-lane, looking only at
// those whose flag bit is set; clears that flag.
__device__ __forceinline__ void warp_drop_max(const unsigned long long (&it)[4], uint32_t& flags) {
    unsigned long long loc = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (((flags >> j) & 1u) && it[j] >= loc) loc = it[j];
    const bool have = flags != 0;
    const uint32_t hi = have ? (uint32_t)(loc >> 32) : 0u;
    const uint32_t mhi = __reduce_max_sync(FULL, hi);
    const uint32_t lo = (have && hi == mhi) ? (uint32_t)loc : 0u;
    const uint32_t mlo = __reduce_max_sync(FULL, lo);
    const unsigned long long worst = ((unsigned long long)mhi << 32) | mlo;
#pragma unroll
    for (int j = 0; j < 4; ++j)
        if (((flags >> j) & 1u) && it[j] == worst) flags &= ~(1u << j);
}

// The W smallest of `count` candidates (W <= count <= CAND_CAP) in ascending order, one per lane:
// a threshold guess selects about W of them (keys are uniform below the scan threshold), a few
// max/min reductions repair the count, the survivors are compacted through `buf` and sorted with
// a 32-lane bitonic network.  Lanes >= W return ~0.
__device__ __forceinline__ unsigned long long warp_top_sorted(unsigned long long* buf, int count, int W,
                                                              uint32_t tinc, int lane) {
    unsigned long long it[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) it[j] = (lane + 32 * j < count) ? buf[lane + 32 * j] : ~0ull;
    __syncwarp();
    const uint32_t guess = (uint32_t)(((unsigned long long)tinc * (unsigned)W) / (unsigned)count);
    uint32_t flags = 0;
    int cnt = 0;
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const bool s = it[j] != ~0ull && (uint32_t)(it[j] >> 32) <= guess;
        if (s) flags |= 1u << j;
        cnt += __popc(__ballot_sync(FULL, s));
    }
    while (cnt > W) {
        warp_drop_max(it, flags);
        --cnt;
    }
    while (cnt < W) {   // add the smallest candidate that is not selected yet
        unsigned long long loc = ~0ull;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (!((flags >> j) & 1u) && it[j] < loc) loc = it[j];
        const uint32_t hi = (uint32_t)(loc >> 32);
        const uint32_t mhi = __reduce_min_sync(FULL, hi);
        const uint32_t lo = (hi == mhi) ? (uint32_t)loc : 0xFFFFFFFFu;
        const uint32_t mlo = __reduce_min_sync(FULL, lo);
        const unsigned long long best = ((unsigned long long)mhi << 32) | mlo;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (!((flags >> j) & 1u) && it[j] == best) flags |= 1u << j;
        ++cnt;
    }
    // compact the W survivors into buf[0..W)
    int base = 0;
    const uint32_t lt = lanemask_lt();
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const bool s = (flags >> j) & 1u;
        const uint32_t b = __ballot_sync(FULL, s);
        if (s) buf[base + __popc(b & lt)] = it[j];
        base += __popc(b);
    }
    __syncwarp();
    unsigned long long x = lane < W ? buf[lane] : ~0ull;
    __syncwarp();
#pragma unroll
    for (int k = 2; k <= 32; k <<= 1) {
#pragma unroll
        for (int j = k >> 1; j > 0; j >>= 1) {
            const unsigned long long other = __shfl_xor_sync(FULL, x, j);
            const bool up = (lane & k) == 0, lower = (lane & j) == 0;
            const bool take_min = (lower == up);
            x = take_min ? (other < x ? other : x) : (other > x ? other : x);
        }
    }
    return x;
}

// First attempt of a refill, split around the neighbour-id loads: issue() extracts the first
// r (+1 spare) candidates in FILL order and starts loading their neighbour ids; settle() uses
// them if they contain r neighbours that are not retained.  Anything else (too few candidates,
// too many, more than one retained neighbour among them) is left to refill_slow().
struct Quick {
    int g;            // candidates whose ids are in flight (0 = attempt unusable)
    uint32_t my_off;
    int32_t my_nb;

    __device__ __forceinline__ void issue(const StepParams& P, int64_t row_start, unsigned long long* buf,
                                          int count, int r, uint32_t tinc, int lane) {
        g = 0;
        my_off = 0;
        my_nb = -1;
        if (count > CAND_CAP || count < r) return;
        if (r >= P.W) {   // full refill: the whole top-W in order, nothing is retained
            g = P.W;
            my_off = (uint32_t)warp_top_sorted(buf, count, P.W, tinc, lane);
            if (lane < g) my_nb = __ldg(P.g.indices + row_start + my_off);
            return;
        }
        unsigned long long it[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) it[j] = (lane + 32 * j < count) ? buf[lane + 32 * j] : ~0ull;
        const int limit = count < P.W ? count : P.W;
        g = (r + 1 < limit) ? r + 1 : limit;
        for (int t = 0; t < g; ++t) {
            const unsigned long long best = warp_pop_min(it);
            if (lane == t) my_off = (uint32_t)best;
        }
        if (lane < g) my_nb = __ldg(P.g.indices + row_start + my_off);
    }

    __device__ __forceinline__ bool settle(const StepParams& P, uint32_t evict_mask, int32_t& slot, int lane) {
        if (g == 0) return false;
        const int r = __popc(evict_mask);
        if (r >= P.W) {   // full refill: candidate t is slot t
            if (lane < P.W) slot = my_nb;
            return true;
        }
        const bool retained = (lane < P.W) && !((evict_mask >> lane) & 1u);
        uint32_t valid = 0;
        for (int t = 0; t < g; ++t) {
            const int32_t x = __shfl_sync(FULL, my_nb, t);
            if (__ballot_sync(FULL, retained && slot == x) == 0) valid |= 1u << t;
        }
        if (__popc(valid) < r) return false;
        const bool ev = (evict_mask >> lane) & 1u;
        const int e = __popc(evict_mask & lanemask_lt());
        const int src = ev ? (int)__fns(valid, 0, e + 1) : 0;
        const int32_t nv = __shfl_sync(FULL, my_nb, src & 31);
        if (ev) slot = nv;
        return true;
    }
};

// Evicted slot mask for this node and step.
__device__ __forceinline__ uint32_t evict_mask_for(const StepParams& P, int32_t v, int lane) {
    const uint32_t wmask = P.W >= 32 ? FULL : ((1u << P.W) - 1u);
    if (P.r >= P.W) return wmask;
    const uint4 o = philox4x32_10_rk((uint32_t)lane >> 2, (uint32_t)v, P.step, P.word_evict, P.rk);
    return warp_smallest_k(word_of(o, lane & 3), wmask, P.r, lane);
}

// First half of S3, fused into the pick: the pick at edge position e claims its id in the relabel table.
__device__ __forceinline__ void register_pick(const StepParams& P, int32_t id, uint32_t n_base, int e) {
    if (P.table) atomicMin(P.table + id, ((unsigned long long)P.stamp << 32) | (n_base + (uint32_t)e));
}

// S2: choose and emit the picks of one node; registers their positions in the relabel table.
__device__ __forceinline__ void warp_pick(const StepParams& P, int32_t v, uint32_t deg, int e_base, uint32_t n_base,
                                          int32_t slot, int lane) {
    const int cnt = deg < (uint32_t)P.W ? (int)deg : P.W;
    const uint32_t cmask = cnt >= 32 ? FULL : ((1u << cnt) - 1u);
    uint32_t pm = cmask;
    if (cnt > P.f) {
        const uint4 o = philox4x32_10_rk((uint32_t)lane >> 2, (uint32_t)v, P.step, P.word_pick, P.rk);
        pm = warp_smallest_k(word_of(o, lane & 3), cmask, P.f, lane);
    }
    if ((pm >> lane) & 1u) {
        const int e = e_base + __popc(pm & lanemask_lt());
        P.picked[e] = slot;
        register_pick(P, slot, n_base, e);
    }
}

// Full Batch Load emission: lanes < cnt hold the chosen neighbour ids; they go out in ascending
// edge offset, which for a sorted CSR row is ascending id.
__device__ __forceinline__ void warp_emit_sorted(const StepParams& P, int cnt, int e_base, uint32_t n_base,
                                                 int32_t id, int lane) {
    int rank = 0;
    for (int t = 0; t < cnt; ++t) {
        const int32_t x = __shfl_sync(FULL, id, t);
        rank += (x < id) ? 1 : 0;
    }
    if (lane < cnt) {
        const int e = e_base + rank;
        P.picked[e] = id;
        register_pick(P, id, n_base, e);
    }
}

// Retry ladder after a failed first attempt: a looser threshold, then the exact scan.
__device__ __noinline__ void refill_slow(const StepParams& P, int32_t v, int64_t row_start, uint32_t deg,
                                         uint32_t evict, unsigned long long* buf, int32_t& slot, int lane) {
    Refill R;
    const uint32_t nq = (deg + 3u) >> 2;
    const int r = __popc(evict);
    if (lane == 0) atomicAdd(P.stats + 0, 1);
    {
        const uint32_t tinc = threshold_for(P.lambda_full, deg);
        const int c = warp_collect(P, v, deg, 0, nq, tinc, buf, 0, lane);
        R.begin(P, row_start, buf, c, tinc == 0xFFFFFFFFu, r, lane);
        __syncwarp();
        if (R.finish(P, row_start, evict, slot, lane)) return;
    }
    warp_exact_top(P, v, deg, buf, lane);
    R.begin(P, row_start, buf, P.W, true, r, lane);
    __syncwarp();
    R.finish(P, row_start, evict, slot, lane);
}

__device__ __forceinline__ void store_row(const StepParams& P, int32_t* row, uint32_t evict, int32_t slot, int lane) {
    if (P.init_rows) {
        if (lane < P.pitch) row[lane] = (lane < P.W) ? slot : -1;
    } else if ((evict >> lane) & 1u) {
        row[lane] = slot;
    }
}

// Registers a hub: reserves an entry and a contiguous range of chunk items with one atomicAdd.
// Returns false if the hub storage is full; the caller then processes the node itself, and the
// part of the reserved item range that exists is marked as holes for the chunk kernel to skip.
// (With hub_degree >= HUB_MIN_DEGREE the storage cannot fill up: the frontier's nodes are
// distinct, so their degrees sum to at most num_edges.)
__device__ __forceinline__ bool hub_register(const StepParams& P, int p, uint32_t deg, int lane) {
    const uint32_t nq = (deg + 3u) >> 2;
    const uint32_t nch = (nq + HUB_CHUNK_QUADS - 1) / HUB_CHUNK_QUADS;
    unsigned long long got = 0;
    if (lane == 0) got = atomicAdd(P.hub_counter, (1ull << 32) | nch);
    got = __shfl_sync(FULL, got, 0);
    const long long h = (long long)(got >> 32);
    const long long cb = (long long)(uint32_t)got;
    const bool ok = h < P.hub_cap && cb + nch <= (long long)P.item_cap;
    if (ok && lane == 0) {
        atomicAdd(P.stats + 1, 1);
        P.hub_entry[h] = make_int2(p, (int)cb);
        P.hub_state[h] = make_int2(0, 0);
    }
    for (long long c = cb + lane; c < cb + nch && c < (long long)P.item_cap; c += 32) P.hub_items[c] = ok ? (int)h : -1;
    return ok;
}

// ---------------------------------------------------------------- warp-per-node kernel
struct NodeState {
    int32_t v;
    int64_t row_start;
    uint32_t deg;
    int e_base;
    int32_t slot;
    uint32_t evict;
    bool refresh, skip, tried_full;
    Quick Q;
};

__global__ void __launch_bounds__(RP_THREADS, 4) k_refresh_pick(const __grid_constant__ StepParams P) {
    chain_wait();
    __shared__ unsigned long long s_buf[RP_WARPS][CAND_CAP];
    if (__ldcg(P.status) != 0) return;   // set only by earlier kernels of the batch: uniform
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned long long* buf = s_buf[wid];
    const int n = P.d_n ? __ldcg(P.d_n) : P.n_host;
    const uint32_t n_base = (uint32_t)n;
    const int refresh_from = P.d_refresh_from ? __ldcg(P.d_refresh_from) : 0;
    const int total_warps = gridDim.x * RP_WARPS;
    int chunk = n / (total_warps * 4);
    chunk = chunk < 1 ? 1 : (chunk > 32 ? 32 : chunk);
    const int W = P.W;

    while (true) {
        int base = 0;
        if (lane == 0) base = atomicAdd(P.work_counter, chunk);
        base = __shfl_sync(FULL, base, 0);
        if (base >= n) break;
        const int cnt = (base + chunk < n ? base + chunk : n) - base;
        // the chunk's node ids, row bounds and pick offsets, one node per lane, all loads in flight together
        int32_t v_l = 0;
        long long lo_l = 0, hi_l = 0;
        int eb_l = 0;
        if (lane < cnt) {
            v_l = P.frontier ? __ldg(P.frontier + base + lane) : base + lane;
            lo_l = __ldg(P.g.indptr + v_l);
            hi_l = __ldg(P.g.indptr + v_l + 1);
            if (P.do_pick) eb_l = __ldg(P.blk_indptr + base + lane);
        }
        // the current cache row of a node (nothing to read when the rows are being initialised)
        auto fetch_row = [&](int i) -> int32_t {
            const int32_t v = __shfl_sync(FULL, v_l, i);
            return (!P.init_rows && !P.fbl && lane < W) ? P.slots[row_offset(P, v) + lane] : -1;
        };
        // nodes of the chunk this kernel has work for: all of them when picking; otherwise (pre-sample,
        // whole-cache refresh) only the rows that need a selection - rows that hold their whole adjacency
        // were written by k_init_low_rows, and the sparse part of a split cache has no rows
        uint32_t todo = __ballot_sync(FULL, lane < cnt && (P.do_pick || hi_l - lo_l > (long long)(P.theta > W ? P.theta : W)));
        auto next_node = [&]() -> int {
            if (!todo) return -1;
            const int b = __ffs(todo) - 1;
            todo &= todo - 1;
            return b;
        };
        int i = next_node();
        int32_t row_next = i >= 0 ? fetch_row(i) : -1;
        NodeState prev;
        prev.skip = true;
        bool have_prev = false;
        while (true) {
            NodeState cur;
            cur.skip = true;
            const bool ran = i >= 0;
            if (ran) {
                const int i_next = next_node();
                // ---- phase A of node i: decide, scan, issue the neighbour-id loads
                cur.v = __shfl_sync(FULL, v_l, i);
                cur.row_start = __shfl_sync(FULL, lo_l, i);
                cur.deg = (uint32_t)(__shfl_sync(FULL, hi_l, i) - cur.row_start);
                cur.e_base = __shfl_sync(FULL, eb_l, i);
                cur.slot = row_next;
                if (i_next >= 0) row_next = fetch_row(i_next);
                cur.skip = false;
                cur.evict = 0;
                cur.tried_full = false;
                cur.Q.g = 0;
                cur.refresh = cur.deg > (uint32_t)W && P.r > 0 && base + i >= refresh_from;
                if (P.fbl && !cur.refresh && lane < (int)cur.deg)   // few neighbours: take them all
                    cur.slot = __ldg(P.g.indices + cur.row_start + lane);
                if (cur.refresh && cur.deg > (uint32_t)P.hub_degree && hub_register(P, base + i, cur.deg, lane)) {
                    cur.skip = true;   // the hub kernel does everything for this node, pick included
                } else if (cur.refresh) {
                    cur.evict = evict_mask_for(P, cur.v, lane);
                    cur.tried_full = !(P.r < W);
                    const uint32_t tinc = threshold_for(cur.tried_full ? P.lambda_full : P.lambda_otf, cur.deg);
                    const int c = warp_collect(P, cur.v, cur.deg, 0, (cur.deg + 3u) >> 2, tinc, buf, 0, lane);
                    cur.Q.issue(P, cur.row_start, buf, c, __popc(cur.evict), tinc, lane);
                    __syncwarp();   // buf may be reused from here on: the first candidates live in registers
                }
                i = i_next;
            }
            if (have_prev && !prev.skip) {
                // ---- phase B of node i-1: its neighbour ids have had a whole scan to arrive
                if (prev.refresh) {
                    if (!prev.Q.settle(P, prev.evict, prev.slot, lane))
                        refill_slow(P, prev.v, prev.row_start, prev.deg, prev.evict, buf, prev.slot, lane);
                    __syncwarp();
                }
                if (P.fbl) {
                    warp_emit_sorted(P, prev.deg < (uint32_t)W ? (int)prev.deg : W, prev.e_base, n_base, prev.slot, lane);
                } else {
                    if (prev.refresh) store_row(P, P.slots + row_offset(P, prev.v), prev.evict, prev.slot, lane);
                    if (P.do_pick) warp_pick(P, prev.v, prev.deg, prev.e_base, n_base, prev.slot, lane);
                }
            }
            prev = cur;
            have_prev = true;
            if (!ran) break;
        }
    }
}

// ---------------------------------------------------------------- warp-per-chunk kernel (hubs)
__global__ void __launch_bounds__(RP_THREADS, 4) k_refresh_pick_hub(const __grid_constant__ StepParams P) {
    chain_wait();
    __shared__ unsigned long long s_buf[RP_WARPS][CAND_CAP];
    if (__ldcg(P.status) != 0) return;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned long long* buf = s_buf[wid];
    const unsigned long long packed = __ldcg(P.hub_counter);
    int total = (int)(uint32_t)packed;
    if (total > P.item_cap) total = P.item_cap;
    if (total == 0) return;
    const uint32_t n_base = (uint32_t)(P.d_n ? __ldcg(P.d_n) : P.n_host);
    const int W = P.W;
    const uint32_t lt = lanemask_lt();
    // a hub's candidates must never run short: its retry would be a serial scan of the whole row
    const float lam = P.r < W ? fmaxf(P.lambda_otf, 32.0f) : P.lambda_full;

    while (true) {
        int w = 0;
        if (lane == 0) w = atomicAdd(P.work_counter2, 1);
        w = __shfl_sync(FULL, w, 0);
        if (w >= total) break;
        const int h = __ldcg(P.hub_items + w);
        if (h < 0) continue;   // a hole left by a hub that did not fit
        const int2 ent = __ldcg(P.hub_entry + h);
        const int p = ent.x;
        const int32_t v = P.frontier ? __ldg(P.frontier + p) : p;
        const long long rs = __ldg(P.g.indptr + v);
        const uint32_t deg = (uint32_t)(__ldg(P.g.indptr + v + 1) - rs);
        const uint32_t nq = (deg + 3u) >> 2;
        const uint32_t nch = (nq + HUB_CHUNK_QUADS - 1) / HUB_CHUNK_QUADS;
        const uint32_t qa = (uint32_t)(w - ent.y) * HUB_CHUNK_QUADS;
        const uint32_t qe = qa + HUB_CHUNK_QUADS < nq ? qa + HUB_CHUNK_QUADS : nq;
        const uint32_t tinc = threshold_for(lam, deg);
        unsigned long long* cand = P.hub_cand + (size_t)h * HUB_CAND_CAP;
        int* cand_count = &P.hub_state[h].x;
        const RowKeys rkeys = philox_row_keys((uint32_t)v, P.step, P.word_fill, P.rk);
        unsigned long long p0 = (unsigned long long)PHILOX_M0 * (unsigned long long)(qa + (uint32_t)lane);
        for (uint32_t qb = qa; qb < qe; qb += 32, p0 = add64(p0, 32ull * PHILOX_M0)) {
            const uint32_t q = qb + lane;
            const uint4 o = philox_row_block(p0, rkeys, P.rk);
            const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
            const bool inq = q < qe;
            const bool any = inq && (__vimin3_u32(min(kk[0], kk[1]), kk[2], kk[3]) <= tinc);
            if (__ballot_sync(FULL, any) == 0) continue;
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const uint32_t off = 4u * q + j;
                const bool hit = inq && (off < deg) && (kk[j] <= tinc);
                const uint32_t b = __ballot_sync(FULL, hit);
                if (b) {
                    int basepos = 0;
                    if (lane == 0) basepos = atomicAdd(cand_count, __popc(b));
                    basepos = __shfl_sync(FULL, basepos, 0);
                    if (hit) {
                        const int pos = basepos + __popc(b & lt);
                        if (pos < HUB_CAND_CAP) cand[pos] = ((unsigned long long)kk[j] << 32) | off;
                    }
                }
            }
        }
        // the warp that finishes the hub's last chunk completes the node
        __threadfence();
        int ticket = 0;
        if (lane == 0) ticket = atomicAdd(&P.hub_state[h].y, 1);
        ticket = __shfl_sync(FULL, ticket, 0);
        if (ticket != (int)nch - 1) continue;
        __threadfence();
        const int c = __ldcg(cand_count);
        for (int j = lane; j < CAND_CAP; j += 32)
            if (j < c) buf[j] = __ldcg(cand + j);
        __syncwarp();
        int32_t* row = P.slots + row_offset(P, v);
        int32_t slot = (!P.init_rows && !P.fbl && lane < W) ? row[lane] : -1;
        const uint32_t evict = evict_mask_for(P, v, lane);
        Quick Q;
        Q.issue(P, rs, buf, c, __popc(evict), tinc, lane);
        __syncwarp();
        if (!Q.settle(P, evict, slot, lane)) refill_slow(P, v, rs, deg, evict, buf, slot, lane);
        __syncwarp();
        if (P.fbl) {
            warp_emit_sorted(P, W, __ldg(P.blk_indptr + p), n_base, slot, lane);
        } else {
            store_row(P, row, evict, slot, lane);
            if (P.do_pick) warp_pick(P, v, deg, __ldg(P.blk_indptr + p), n_base, slot, lane);
        }
    }
}

// ================================================================ split OTF path
// For a partial refresh (0 < r < W) the work is split in two kernels:
//   k_scan    one warp per work item (a 4096-offset chunk of one refreshed node): nothing but
//             Philox blocks and a threshold compare, at full occupancy; the few offsets below the
//             threshold go to the node's candidate list in global memory (at most 64, two per lane).
//   k_finish  one warp per frontier node: eviction, refill from the candidate list, row update
//             and the pick.  Rows of up to SMALL_DEGREE neighbours skip the scan: one Philox block
//             per lane covers the whole row, and the refill is decided in registers.
// Nodes whose candidate list cannot decide the refill (too few, too many, or several retained
// neighbours among the first ones) take the retry ladder of the fused path.

__global__ void __launch_bounds__(RP_THREADS, GS_SCAN_MIN_BLOCKS) k_scan(const __grid_constant__ StepParams P) {
    chain_wait();
    __shared__ unsigned long long s_stage[RP_WARPS][SPLIT_CAND_CAP];
    __shared__ int s_hits[RP_WARPS];
    if (__ldcg(P.status) != 0) return;
    const int lane = threadIdx.x & 31;
    unsigned long long* stage = s_stage[threadIdx.x >> 5];
    int* hits = &s_hits[threadIdx.x >> 5];
    const int total = __ldcg(P.d_items_total);
    const int total_warps = gridDim.x * RP_WARPS;
    // Work is handed out in batches of 1..32 items; every warp owns one batch up front, the rest
    // goes through the shared counter.
    int batch = total / (total_warps * GS_SCAN_BATCH_DIV);
    batch = batch < 1 ? 1 : (batch > 32 ? 32 : batch);
    const uint32_t lt = lanemask_lt();
    const int warp_gid = blockIdx.x * RP_WARPS + (threadIdx.x >> 5);
    // every warp owns one batch up front; the next one is asked for while the current one is scanned, so the
    // round trip of the atomic is never waited for
    int base = warp_gid * batch;
    while (base < total) {
        int next_base = 0;
        if (lane == 0) next_base = atomicAdd(P.work_counter_scan, batch) + total_warps * batch;
        const int cnt = (base + batch < total ? base + batch : total) - base;
        int4 d_l = make_int4(0, 0, 0, 0);
        if (lane < cnt) d_l = __ldg(P.items + base + lane);
        for (int i = 0; i < cnt; ++i) {
            const int p = __shfl_sync(FULL, d_l.x, i);
            const int32_t v = __shfl_sync(FULL, d_l.y, i);
            const uint32_t deg = (uint32_t)__shfl_sync(FULL, d_l.z, i);
            const int chunk = __shfl_sync(FULL, d_l.w, i);
            const uint32_t nq = (deg + 3u) >> 2;
            const bool single = nq <= (uint32_t)HUB_CHUNK_QUADS;
            const uint32_t qa = (uint32_t)chunk * HUB_CHUNK_QUADS;
            const uint32_t qe = qa + HUB_CHUNK_QUADS < nq ? qa + HUB_CHUNK_QUADS : nq;
            const uint32_t tinc = threshold_for(P.lambda_otf, deg);
            // Hits of this item are staged in shared memory; each hitting lane reserves its place with a
            // shared-memory atomic (hits are rare, the order inside the list does not matter), so an
            // iteration with hits costs a few instructions, not a vote per key.  Hits beyond the cap
            // are only counted.
            if (lane == 0) *hits = 0;
            __syncwarp();
            auto take_hits = [&](uint32_t q, const uint4& o, bool inq) {
                const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
                if (!inq || min(min(kk[0], kk[1]), min(kk[2], kk[3])) > tinc) return;
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    const uint32_t off = 4u * q + j;
                    if (off < deg && kk[j] <= tinc) {
                        const int pos = atomicAdd(hits, 1);
                        if (pos < SPLIT_CAND_CAP) stage[pos] = ((unsigned long long)kk[j] << 32) | off;
                    }
                }
            };
            // Main loop: four independent Philox blocks per lane and iteration (512 offsets per warp
            // iteration), all quads in range, one vote per iteration.  The ragged end takes up to four
            // masked blocks at once as well.
            // the row's quads share the first two Philox rounds' constants; M0 * q advances by adds
            const RowKeys rkeys = philox_row_keys((uint32_t)v, P.step, P.word_fill, P.rk);
            constexpr unsigned long long M0x32 = 32ull * PHILOX_M0;
            unsigned long long p0 = (unsigned long long)PHILOX_M0 * (unsigned long long)(qa + (uint32_t)lane);
            uint32_t qb = qa;
            for (; qb + 128 <= qe; qb += 128, p0 = add64(p0, 4 * M0x32)) {
                const uint32_t q = qb + lane;
                const uint4 o0 = philox_row_block(p0, rkeys, P.rk);
                const uint4 o1 = philox_row_block(add64(p0, M0x32), rkeys, P.rk);
                const uint4 o2 = philox_row_block(add64(p0, 2 * M0x32), rkeys, P.rk);
                const uint4 o3 = philox_row_block(add64(p0, 3 * M0x32), rkeys, P.rk);
                // the smallest of the 16 keys with three-input minima: 8 instructions instead of 15
                const uint32_t m0 = __vimin3_u32(o0.x, o0.y, o0.z), m1 = __vimin3_u32(o1.x, o1.y, o1.z);
                const uint32_t m2 = __vimin3_u32(o2.x, o2.y, o2.z), m3 = __vimin3_u32(o3.x, o3.y, o3.z);
                const uint32_t ma = __vimin3_u32(m0, o0.w, o1.w), mb = __vimin3_u32(m1, o2.w, o3.w);
                if (__ballot_sync(FULL, min(__vimin3_u32(ma, mb, m2), m3) <= tinc) == 0) continue;
                take_hits(q, o0, true);
                take_hits(q + 32, o1, true);
                take_hits(q + 64, o2, true);
                take_hits(q + 96, o3, true);
            }
            if (qb < qe) {
                const uint32_t q = qb + lane;
                const int groups = (int)((qe - qb + 31u) >> 5);   // 1..4 groups of 32 quads remain
                if (groups > 2) {
                    const uint4 o0 = philox_row_block(p0, rkeys, P.rk);
                    const uint4 o1 = philox_row_block(add64(p0, M0x32), rkeys, P.rk);
                    const uint4 o2 = philox_row_block(add64(p0, 2 * M0x32), rkeys, P.rk);
                    take_hits(q, o0, q < qe);
                    take_hits(q + 32, o1, q + 32 < qe);
                    take_hits(q + 64, o2, q + 64 < qe);
                    if (groups > 3) {
                        const uint4 o3 = philox_row_block(add64(p0, 3 * M0x32), rkeys, P.rk);
                        take_hits(q + 96, o3, q + 96 < qe);
                    }
                } else {
                    const uint4 o0 = philox_row_block(p0, rkeys, P.rk);
                    take_hits(q, o0, q < qe);
                    if (groups > 1) {
                        const uint4 o1 = philox_row_block(add64(p0, M0x32), rkeys, P.rk);
                        take_hits(q + 32, o1, q + 32 < qe);
                    }
                }
            }
            __syncwarp();
            const int count = *hits;
            __syncwarp();
            // publish: the only warp of a short row owns the list; the chunks of a long row reserve
            // their range with one atomic per chunk, so no warp waits on an atomic inside the scan
            int dst = 0;
            if (single) {
                if (lane == 0) P.cand_count[p] = count;
            } else if (count > 0) {
                if (lane == 0) dst = atomicAdd(P.cand_count + p, count);
                dst = __shfl_sync(FULL, dst, 0);
            }
            for (int t = lane; t < count && t < SPLIT_CAND_CAP; t += 32)
                if (dst + t < SPLIT_CAND_CAP) P.cand[(size_t)p * SPLIT_CAND_CAP + dst + t] = stage[t];
            __syncwarp();
        }
        base = __shfl_sync(FULL, next_base, 0);
    }
}

// EVICT keys (lanes 0-7 compute the eight slot quads) and PICK keys (lanes 8-15) from one Philox call.
__device__ __forceinline__ void evict_pick_keys(const StepParams& P, int32_t v, int lane, uint32_t& ekey,
                                                uint32_t& pkey) {
    const bool second = (lane >> 3) & 1;
    const uint4 o = philox4x32_10_rk((uint32_t)lane & 7u, (uint32_t)v, P.step, second ? P.word_pick : P.word_evict, P.rk);
    const int src = lane >> 2, w = lane & 3;
    const uint32_t e0 = __shfl_sync(FULL, o.x, src), e1 = __shfl_sync(FULL, o.y, src);
    const uint32_t e2 = __shfl_sync(FULL, o.z, src), e3 = __shfl_sync(FULL, o.w, src);
    const uint32_t p0 = __shfl_sync(FULL, o.x, src + 8), p1 = __shfl_sync(FULL, o.y, src + 8);
    const uint32_t p2 = __shfl_sync(FULL, o.z, src + 8), p3 = __shfl_sync(FULL, o.w, src + 8);
    ekey = w == 0 ? e0 : (w == 1 ? e1 : (w == 2 ? e2 : e3));
    pkey = w == 0 ? p0 : (w == 1 ? p1 : (w == 2 ? p2 : p3));
}

// Refill of a row with at most SMALL_DEGREE neighbours, decided in registers: lane l holds offsets
// 4l..4l+3 with their keys and neighbour ids; offsets whose neighbour is retained are struck out
// and the r smallest remaining (key, offset) pairs go to the evicted slots in ascending order.
__device__ __forceinline__ void small_refill(const StepParams& P, int32_t v, int64_t row_start, uint32_t deg,
                                             uint32_t evict, int32_t& slot, int lane) {
    const uint4 o = philox4x32_10_rk((uint32_t)lane, (uint32_t)v, P.step, P.word_fill, P.rk);
    const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
    int32_t nb[4];
    bool ok[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) {
        const uint32_t off = 4u * lane + j;
        ok[j] = off < deg;
        nb[j] = ok[j] ? __ldg(P.g.indices + row_start + off) : -1;
    }
    const uint32_t wmask = P.W >= 32 ? FULL : ((1u << P.W) - 1u);
    uint32_t rm = wmask & ~evict;
    while (rm) {
        const int t = __ffs(rm) - 1;
        rm &= rm - 1;
        const int32_t s = __shfl_sync(FULL, slot, t);
#pragma unroll
        for (int j = 0; j < 4; ++j) ok[j] = ok[j] && nb[j] != s;
    }
    unsigned long long it[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) it[j] = ok[j] ? (((unsigned long long)kk[j] << 32) | (4u * lane + j)) : ~0ull;
    uint32_t em = evict;
    while (em) {
        const int dst = __ffs(em) - 1;
        em &= em - 1;
        unsigned long long before[4];
#pragma unroll
        for (int j = 0; j < 4; ++j) before[j] = it[j];
        const unsigned long long best = warp_pop_min(it);
        int32_t mine = -1;
#pragma unroll
        for (int j = 0; j < 4; ++j)
            if (before[j] == best) mine = nb[j];
        const uint32_t owner = __ballot_sync(FULL, mine >= 0);
        const int32_t nv = __shfl_sync(FULL, mine, __ffs(owner) - 1);
        if (lane == dst) slot = nv;
    }
}

__global__ void __launch_bounds__(RP_THREADS, GS_FINISH_MIN_BLOCKS) k_finish(const __grid_constant__ StepParams P) {
    chain_wait();
    __shared__ unsigned long long s_buf[RP_WARPS][CAND_CAP];
    if (__ldcg(P.status) != 0) return;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned long long* buf = s_buf[wid];
    const int n = __ldcg(P.d_n);
    const uint32_t n_base = (uint32_t)n;
    const int refresh_from = P.d_refresh_from ? __ldcg(P.d_refresh_from) : 0;
    const int total_warps = gridDim.x * RP_WARPS;
    int chunk = n / (total_warps * 2);
    chunk = chunk < 4 ? 4 : (chunk > 32 ? 32 : chunk);
    const int W = P.W;
    const uint32_t wmask = W >= 32 ? FULL : ((1u << W) - 1u);
    const int warp_gid = blockIdx.x * RP_WARPS + wid;
    bool first_grab = true;   // one chunk per warp is assigned statically, the rest through the counter

    while (true) {
        int base = 0;
        if (first_grab) {
            base = warp_gid * chunk;
            first_grab = false;
        } else {
            if (lane == 0) base = atomicAdd(P.work_counter, chunk) + total_warps * chunk;
            base = __shfl_sync(FULL, base, 0);
        }
        if (base >= n) break;
        const int cnt = (base + chunk < n ? base + chunk : n) - base;
        int32_t v_l = 0;
        long long lo_l = 0, hi_l = 0;
        int eb_l = 0, cc_l = 0;
        if (lane < cnt) {
            v_l = __ldg(P.frontier + base + lane);
            lo_l = __ldg(P.g.indptr + v_l);
            hi_l = __ldg(P.g.indptr + v_l + 1);
            eb_l = __ldg(P.blk_indptr + base + lane);
            cc_l = __ldcg(P.cand_count + base + lane);
        }
        // one node ahead: its cache row and its candidate list are in flight while this one is decided
        int32_t row_next = -1;
        unsigned long long cand_next = ~0ull, cand_next2 = ~0ull;
        auto prefetch = [&](int i) {
            const int32_t v = __shfl_sync(FULL, v_l, i);
            const int cc = __shfl_sync(FULL, cc_l, i);
            const int64_t ro = P.fbl ? -1 : row_offset(P, v);
            row_next = (ro >= 0 && lane < W) ? P.slots[ro + lane] : -1;
            const unsigned long long* cl = P.cand + (size_t)(base + i) * SPLIT_CAND_CAP;
            cand_next = (lane < cc) ? __ldcg(cl + lane) : ~0ull;
            cand_next2 = (lane + 32 < cc && lane + 32 < SPLIT_CAND_CAP) ? __ldcg(cl + lane + 32) : ~0ull;
        };
        prefetch(0);
        for (int i = 0; i < cnt; ++i) {
            const int p = base + i;
            const int32_t v = __shfl_sync(FULL, v_l, i);
            const int64_t rs = __shfl_sync(FULL, lo_l, i);
            const uint32_t deg = (uint32_t)(__shfl_sync(FULL, hi_l, i) - rs);
            const int e_base = __shfl_sync(FULL, eb_l, i);
            const int cc = __shfl_sync(FULL, cc_l, i);
            int32_t slot = row_next;
            unsigned long long cand = cand_next, cand2 = cand_next2;
            if (i + 1 < cnt) prefetch(i + 1);
            const bool refresh = deg > (uint32_t)W && P.r > 0 && p >= refresh_from;
            const int ncached = deg < (uint32_t)W ? (int)deg : W;
            if (!P.fbl && P.theta >= 0 && deg <= (uint32_t)P.theta) {
                // Sparse part of a split cache (degree <= theta <= SMALL_DEGREE): no cache row exists;
                // the node is sampled from the graph by the Full Batch Load rule, in every mode.
                const int f = P.f;
                int32_t id = -1;
                if ((int)deg <= f) {
                    if (lane < (int)deg) id = __ldg(P.g.indices + rs + lane);
                } else {
                    const uint4 o = philox4x32_10_rk((uint32_t)lane, (uint32_t)v, P.step, P.word_fetch, P.rk);
                    const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (4u * lane + j < deg) buf[4 * lane + j] = ((unsigned long long)kk[j] << 32) | (4u * lane + j);
                    __syncwarp();
                    const unsigned long long x = warp_top_sorted(buf, (int)deg, f, 0xFFFFFFFFu, lane);
                    if (lane < f) id = __ldg(P.g.indices + rs + (uint32_t)x);
                    __syncwarp();
                }
                warp_emit_sorted(P, (int)deg < f ? (int)deg : f, e_base, n_base, id, lane);
                continue;
            }
            if (P.fbl && !refresh) {
                // Full Batch Load of a short row: the whole adjacency, already in ascending offset
                if (lane < (int)deg) {
                    const int32_t id = __ldg(P.g.indices + rs + lane);
                    const int e = e_base + lane;
                    P.picked[e] = id;
                    register_pick(P, id, n_base, e);
                }
                continue;
            }
            uint32_t ekey = 0, pkey = 0;
            if (!P.fbl && (refresh || ncached > P.f)) evict_pick_keys(P, v, lane, ekey, pkey);
            uint32_t cache_part = 0;   // OTF Fetch: lanes of the cache slots that are part of the sample
            if (refresh && P.r >= W && !P.fetch) {
                // Full refill (FCR, and Full Batch Load with W = f): the W offsets first in key order,
                // in that order.  Short rows take every offset as a candidate, longer ones the list
                // the scan kernel left; a list that cannot hold the top-W sends the row to a rescan.
                int c = -1;
                uint32_t tinc = 0xFFFFFFFFu;
                if (deg <= (uint32_t)SMALL_DEGREE) {
                    const uint4 o = philox4x32_10_rk((uint32_t)lane, (uint32_t)v, P.step, P.word_fill, P.rk);
                    const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                    for (int j = 0; j < 4; ++j)
                        if (4u * lane + j < deg) buf[4 * lane + j] = ((unsigned long long)kk[j] << 32) | (4u * lane + j);
                    c = (int)deg;
                } else if (cc >= W && cc <= SPLIT_CAND_CAP) {
                    if (lane < cc) buf[lane] = cand;
                    if (lane + 32 < cc) buf[lane + 32] = cand2;
                    c = cc;
                    tinc = threshold_for(P.lambda_otf, deg);
                }
                __syncwarp();
                if (c >= W) {
                    const unsigned long long x = warp_top_sorted(buf, c, W, tinc, lane);
                    slot = lane < W ? __ldg(P.g.indices + rs + (uint32_t)x) : -1;
                    __syncwarp();
                } else {
                    if (deg > (uint32_t)RETRY_QUEUE_DEGREE && hub_register(P, p, deg, lane)) continue;
                    refill_slow(P, v, rs, deg, wmask, buf, slot, lane);
                    __syncwarp();
                }
                if (P.fbl) {
                    warp_emit_sorted(P, W, e_base, n_base, slot, lane);
                    continue;
                }
                if (lane < W) P.slots[row_offset(P, v) + lane] = slot;
            } else if (refresh) {
                uint32_t evict;
                if (P.fetch) {
                    // (OTF Fetch comes here even when all f = W samples are fetched: it never writes the row.)
                    // The f - r cache picks play the part of the retained slots, the r fetched
                    // neighbours land in the r lowest other lanes; the other slots are blanked so that
                    // only the cache picks exclude candidates.  The row itself is not modified.
                    cache_part = warp_smallest_k(pkey, wmask, P.f - P.r, lane);
                    const uint32_t rest = wmask & ~cache_part;
                    const bool mine = ((rest >> lane) & 1u) && __popc(rest & lanemask_lt()) < P.r;
                    evict = __ballot_sync(FULL, mine);
                    if (!((cache_part >> lane) & 1u)) slot = -1;
                } else {
                    evict = warp_smallest_k(ekey, wmask, P.r, lane);
                }
                if (deg <= (uint32_t)SMALL_DEGREE) {
                    small_refill(P, v, rs, deg, evict, slot, lane);
                } else {
                    bool done = false;
                    if (cc >= P.r && cc <= SPLIT_CAND_CAP) {
                        // Candidates are taken in FILL order, a few at a time, until r of them are not
                        // retained neighbours; lane t keeps the t-th candidate.  Never more than the
                        // first W matter (refill rule), so W lanes are enough.
                        const int limit = cc < W ? cc : W;
                        const bool retained = (lane < W) && !((evict >> lane) & 1u);
                        int taken = 0;
                        int g = P.r + (deg < 1024u ? 4 : 1);
                        uint32_t my_off = 0, valid = 0;
                        int32_t my_nb = -1;
                        while (true) {
                            g = g < limit - taken ? g : limit - taken;
                            for (int t = taken; t < taken + g; ++t) {
                                const unsigned long long loc = cand < cand2 ? cand : cand2;
                                const uint32_t hi = (uint32_t)(loc >> 32);
                                const uint32_t mhi = __reduce_min_sync(FULL, hi);
                                const uint32_t lo = (hi == mhi) ? (uint32_t)loc : 0xFFFFFFFFu;
                                const uint32_t mlo = __reduce_min_sync(FULL, lo);
                                const unsigned long long best = ((unsigned long long)mhi << 32) | mlo;
                                if (cand == best) cand = ~0ull;
                                if (cand2 == best) cand2 = ~0ull;
                                if (lane == t) my_off = mlo;
                            }
                            if (lane >= taken && lane < taken + g) my_nb = __ldg(P.g.indices + rs + my_off);
                            for (int t = taken; t < taken + g; ++t) {
                                const int32_t x = __shfl_sync(FULL, my_nb, t);
                                if (__ballot_sync(FULL, retained && slot == x) == 0) valid |= 1u << t;
                            }
                            taken += g;
                            if (__popc(valid) >= P.r || taken >= limit) break;
                            g = P.r - __popc(valid) + 1;
                        }
                        // enough winners, or the whole top-W was examined (which cannot lack winners);
                        // a list shorter than W that ran dry decides nothing and the row is rescanned
                        if (__popc(valid) >= P.r) {
                            // t-th valid candidate -> t-th evicted slot, through shared memory
                            const int vr = __popc(valid & lanemask_lt());
                            int32_t* stage = reinterpret_cast<int32_t*>(buf);
                            if (((valid >> lane) & 1u) && vr < P.r) stage[vr] = my_nb;
                            __syncwarp();
                            if ((evict >> lane) & 1u) slot = stage[__popc(evict & lanemask_lt())];
                            __syncwarp();
                            done = true;
                        }
                    }
                    if (!done) {
                        // A long row is not rescanned by this one warp: it is queued for the chunked
                        // hub kernel, which redoes the node (pick included) with all warps.
                        if (!P.fetch && deg > (uint32_t)RETRY_QUEUE_DEGREE && hub_register(P, p, deg, lane)) continue;
                        refill_slow(P, v, rs, deg, evict, buf, slot, lane);
                        __syncwarp();
                    }
                }
                if (P.fetch) {
                    // emit the cache part in ascending slot index, then the fetched part in FETCH order
                    const uint32_t lt = lanemask_lt();
                    int e = -1;
                    if ((cache_part >> lane) & 1u) e = e_base + __popc(cache_part & lt);
                    else if ((evict >> lane) & 1u) e = e_base + (P.f - P.r) + __popc(evict & lt);
                    if (e >= 0) {
                        P.picked[e] = slot;
                        register_pick(P, slot, n_base, e);
                    }
                    continue;
                }
                if ((evict >> lane) & 1u) P.slots[row_offset(P, v) + lane] = slot;
            }
            // S2 pick
            const uint32_t cmask = ncached >= 32 ? FULL : ((1u << ncached) - 1u);
            uint32_t pm = cmask;
            if (ncached > P.f) pm = warp_smallest_k(pkey, cmask, P.f, lane);
            if ((pm >> lane) & 1u) {
                const int e = e_base + __popc(pm & lanemask_lt());
                P.picked[e] = slot;
                register_pick(P, slot, n_base, e);
            }
        }
    }
}

cudaError_t launch_scan(const StepParams& p, int64_t item_bound, cudaStream_t s) {
    // the blocks that are resident together walk all the work: a block that only starts when another one has
    // left would find its up-front batch late, at the tail of the launch
    static int resident = 0;   // same kernel, same block size on every device of a process
    if (resident <= 0) {
        int r = 0;
        if (cudaOccupancyMaxActiveBlocksPerMultiprocessor(&r, k_scan, RP_THREADS, 0) != cudaSuccess || r < 1) r = 2;
        resident = r;
    }
    const int64_t cap = sm_count() * resident;
    int64_t sb = (item_bound + RP_WARPS - 1) / RP_WARPS;
    sb = limit_grid(sb > cap ? cap : (sb < 1 ? 1 : sb));
    launch_chained(k_scan, sb, RP_THREADS, s, p);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_finish(const StepParams& p, int64_t n_bound, cudaStream_t s) {
    const int64_t cap = sm_count() * 8;
    int64_t fb = (n_bound + RP_WARPS - 1) / RP_WARPS;
    fb = limit_grid(fb > cap ? cap : (fb < 1 ? 1 : fb));
    launch_chained(k_finish, fb, RP_THREADS, s, p);
    int launched = 1;
    if (p.hub_cap > 0) {   // rows queued for a rescan; exits at once when there are none
        // a partial refresh queues a handful of rows per batch at most, a full one about 1 % of them
        const int64_t hub_grid = limit_grid((p.r >= p.W) ? cap : sm_count() * 2);
        launch_chained(k_refresh_pick_hub, hub_grid, RP_THREADS, s, p);
        launched = 2;
    }
    count_launches(launched);
    return cudaGetLastError();
}

// S0 for rows that hold their whole adjacency (deg <= W): slot j = j-th neighbour in CSR order, -1
// beyond; the same row goes to every cache.  One thread per slot, fully coalesced stores.
__global__ void __launch_bounds__(256) k_init_low_rows(GraphView g, int32_t* slots, int pitch, int W, int caches) {
    const int64_t total = g.num_nodes * (int64_t)pitch;
    const int64_t cache_stride = total;
    for (int64_t idx = (int64_t)blockIdx.x * blockDim.x + threadIdx.x; idx < total; idx += (int64_t)gridDim.x * blockDim.x) {
        const int64_t v = idx / pitch;
        const int j = (int)(idx - v * pitch);
        const long long rs = __ldg(g.indptr + v);
        const long long deg = __ldg(g.indptr + v + 1) - rs;
        if (deg > (long long)W) continue;
        const int32_t val = (j < (int)deg) ? __ldg(g.indices + rs + j) : -1;
        for (int c = 0; c < caches; ++c) __stcs(slots + c * cache_stride + idx, val);
    }
}

cudaError_t launch_init_low_rows(const GraphView& g, int32_t* slots, int32_t pitch, int32_t W, int32_t caches,
                                 cudaStream_t s) {
    k_init_low_rows<<<(int)(sm_count() * 16), 256, 0, s>>>(g, slots, pitch, W, caches);
    count_launches(1);
    return cudaGetLastError();
}

cudaError_t launch_refresh_pick(const StepParams& p, int64_t n_bound, cudaStream_t s) {
    int64_t blocks = (n_bound + RP_WARPS - 1) / RP_WARPS;
    const int64_t cap = sm_count() * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    blocks = limit_grid(blocks);
    launch_chained(k_refresh_pick, blocks, RP_THREADS, s, p);
    int launched = 1;
    if (p.hub_cap > 0) {
        launch_chained(k_refresh_pick_hub, limit_grid(cap), RP_THREADS, s, p);
        launched = 2;
    }
    count_launches(launched);
    return cudaGetLastError();
}

}  // namespace gs
