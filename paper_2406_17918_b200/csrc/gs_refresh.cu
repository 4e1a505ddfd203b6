// S0 static pre-sample, S1 refresh (FCR / OTF) and S2 pick, fused per frontier node.
//
// Every selection is "the k items first in (key, index) order" with Philox keys that depend on
// (node, item index, step) only - not on the neighbour ids.  The scan over a node's deg edge
// offsets therefore reads no CSR bytes: it evaluates one Philox block per four offsets, keeps the
// offsets whose key is below a threshold chosen so that about lambda of them survive, and only
// then reads the few neighbour ids it needs.  If the survivors turn out not to be enough (or
// too many for the buffer) the node is redone with a larger lambda and finally with an exact
// running top-W, so the result never depends on the threshold.
//
// Refill rule used (it follows from the refresh definition): the r refill winners are the first r
// entries, after removing retained neighbours, of the top-W list of ALL edge offsets in FILL
// order, because at most W - r retained neighbours can precede the r-th winner.
#include "gs_device.cuh"
#include "gs_internal.h"

namespace gs {

constexpr int RP_THREADS = 256;         // warp-per-node kernel
constexpr int RP_WARPS = RP_THREADS / 32;
constexpr int HUB_THREADS = 512;        // block-per-node kernel

struct NodeCtx {
    int32_t v;
    int64_t row_start;
    uint32_t deg;
};

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
    for (uint32_t qb = q_begin; qb < q_end; qb += 32) {
        const uint32_t q = qb + lane;
        const uint4 o = philox4x32_10(q, (uint32_t)v, P.step, P.word_fill, P.key0, P.key1);
        const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const uint32_t off = 4u * q + w;
            const bool hit = (q < q_end) && (off < deg) && (kk[w] <= tinc);
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
    return count;
}

// Exact fallback: one warp keeps the W smallest (key, offset) pairs in a sorted list, one per
// lane, while scanning every offset.  Leaves them in buf[0..W) in order.
__device__ void warp_exact_top(const StepParams& P, int32_t v, uint32_t deg, unsigned long long* buf, int lane) {
    const int W = P.W;
    unsigned long long cur = ~0ull;
    const uint32_t nq = (deg + 3u) >> 2;
    for (uint32_t qb = 0; qb < nq; qb += 32) {
        const uint32_t q = qb + lane;
        const uint4 o = philox4x32_10(q, (uint32_t)v, P.step, P.word_fill, P.key0, P.key1);
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

// One warp: given c candidates in buf (all offsets with key <= threshold; `whole` = they are all
// the offsets, or at least the exact top-W), fill the evicted slots.  Returns false if the
// candidates cannot decide the refill (caller retries with more).
__device__ bool warp_refill(const StepParams& P, const NodeCtx& nd, const unsigned long long* buf, int c,
                            bool whole, uint32_t evict_mask, int32_t& slot, int lane) {
    const int W = P.W;
    const int r = __popc(evict_mask);
    if (c > CAND_CAP) return false;
    if (c < r) return false;
    unsigned long long it[4];
#pragma unroll
    for (int j = 0; j < 4; ++j) it[j] = (lane + 32 * j < c) ? buf[lane + 32 * j] : ~0ull;
    const int limit = c < W ? c : W;          // never more than the top-W matter
    const bool retained = (lane < W) && !((evict_mask >> lane) & 1u);
    int taken = 0;
    uint32_t valid = 0;
    uint32_t my_off = 0;
    int32_t my_nb = -1;
    while (true) {
        int g = r - __popc(valid);
        if (g > limit - taken) g = limit - taken;
        for (int t = 0; t < g; ++t) {
            const unsigned long long best = warp_pop_min(it);
            if (lane == taken + t) my_off = (uint32_t)best;
        }
        if (lane >= taken && lane < taken + g) my_nb = P.g.indices[nd.row_start + my_off];
        for (int t = taken; t < taken + g; ++t) {
            const int32_t x = __shfl_sync(FULL, my_nb, t);
            const uint32_t hit = __ballot_sync(FULL, retained && slot == x);
            if (hit == 0) valid |= 1u << t;
        }
        taken += g;
        if (__popc(valid) >= r) break;
        if (taken >= limit) {
            // candidates exhausted: only conclusive if they covered the whole top-W
            if (whole || c >= W) break;  // cannot happen with fewer than r valid (refill rule)
            return false;
        }
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

// Evicted slot mask for this node and step.
__device__ __forceinline__ uint32_t evict_mask_for(const StepParams& P, int32_t v, int lane) {
    const uint32_t wmask = P.W >= 32 ? FULL : ((1u << P.W) - 1u);
    if (P.r >= P.W) return wmask;
    const uint4 o = philox4x32_10((uint32_t)lane >> 2, (uint32_t)v, P.step, P.word_evict, P.key0, P.key1);
    return warp_smallest_k(word_of(o, lane & 3), wmask, P.r, lane);
}

// S2: choose and emit the picks of one node; registers their positions in the relabel table.
__device__ __forceinline__ void warp_pick(const StepParams& P, const NodeCtx& nd, int p, int32_t slot, int lane) {
    const int cnt = nd.deg < (uint32_t)P.W ? (int)nd.deg : P.W;
    const uint32_t cmask = cnt >= 32 ? FULL : ((1u << cnt) - 1u);
    uint32_t pm = cmask;
    if (cnt > P.f) {
        const uint4 o = philox4x32_10((uint32_t)lane >> 2, (uint32_t)nd.v, P.step, P.word_pick, P.key0, P.key1);
        pm = warp_smallest_k(word_of(o, lane & 3), cmask, P.f, lane);
    }
    if ((pm >> lane) & 1u) {
        const int e = P.blk_indptr[p] + __popc(pm & lanemask_lt());
        P.picked[e] = slot;
        const uint32_t n = (uint32_t)__ldcg(P.d_n);
        atomicMin(P.table + slot, ((unsigned long long)P.stamp << 32) | (n + (uint32_t)e));
    }
}

__device__ __forceinline__ bool load_node(const StepParams& P, int p, NodeCtx& nd, int lane) {
    int32_t v = P.frontier ? P.frontier[p] : p;
    long long a = 0;
    if (lane < 2) a = P.g.indptr[v + lane];
    const long long rs = __shfl_sync(FULL, a, 0);
    const long long re = __shfl_sync(FULL, a, 1);
    nd.v = v;
    nd.row_start = rs;
    nd.deg = (uint32_t)(re - rs);
    return true;
}

// ---------------------------------------------------------------- warp-per-node kernel
__global__ void __launch_bounds__(RP_THREADS) k_refresh_pick(StepParams P) {
    __shared__ unsigned long long s_buf[RP_WARPS][CAND_CAP];
    if (__ldcg(P.status) != 0) return;   // set only by earlier kernels of the batch: uniform
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    unsigned long long* buf = s_buf[wid];
    const int n = P.d_n ? __ldcg(P.d_n) : P.n_host;
    const int refresh_from = P.d_refresh_from ? __ldcg(P.d_refresh_from) : 0;
    const int total_warps = gridDim.x * RP_WARPS;
    int chunk = n / (total_warps * 8);
    chunk = chunk < 1 ? 1 : (chunk > 64 ? 64 : chunk);
    const int W = P.W;

    while (true) {
        int base = 0;
        if (lane == 0) base = atomicAdd(P.work_counter, chunk);
        base = __shfl_sync(FULL, base, 0);
        if (base >= n) break;
        const int end = base + chunk < n ? base + chunk : n;
        for (int p = base; p < end; ++p) {
            NodeCtx nd;
            load_node(P, p, nd, lane);
            int32_t* row = P.slots + (int64_t)nd.v * P.pitch;
            int32_t slot = -1;
            if (P.init_rows) {
                if (nd.deg <= (uint32_t)W) {
                    if (lane < (int)nd.deg) slot = P.g.indices[nd.row_start + lane];
                    if (lane < P.pitch) row[lane] = slot;
                }
            } else if (lane < W) {
                slot = row[lane];
            }
            const bool refresh = nd.deg > (uint32_t)W && P.r > 0 && p >= refresh_from;
            if (refresh) {
                if (nd.deg > (uint32_t)P.hub_degree) {   // a whole block handles this one, pick included
                    if (lane == 0) P.hub_list[atomicAdd(P.hub_count, 1)] = p;
                    continue;
                }
                const uint32_t evict = evict_mask_for(P, nd.v, lane);
                const uint32_t nq = (nd.deg + 3u) >> 2;
                bool done = false;
                if (P.r < W) {
                    const uint32_t tinc = threshold_for(P.lambda_otf, nd.deg);
                    const int c = warp_collect(P, nd.v, nd.deg, 0, nq, tinc, buf, 0, lane);
                    __syncwarp();
                    done = warp_refill(P, nd, buf, c, tinc == 0xFFFFFFFFu, evict, slot, lane);
                    __syncwarp();
                }
                if (!done) {
                    const uint32_t tinc = threshold_for(P.lambda_full, nd.deg);
                    const int c = warp_collect(P, nd.v, nd.deg, 0, nq, tinc, buf, 0, lane);
                    __syncwarp();
                    done = warp_refill(P, nd, buf, c, tinc == 0xFFFFFFFFu, evict, slot, lane);
                    __syncwarp();
                }
                if (!done) {
                    warp_exact_top(P, nd.v, nd.deg, buf, lane);
                    warp_refill(P, nd, buf, W, true, evict, slot, lane);
                    __syncwarp();
                }
                if (P.init_rows) {
                    if (lane < P.pitch) row[lane] = (lane < W) ? slot : -1;
                } else if ((evict >> lane) & 1u) {
                    row[lane] = slot;
                }
            }
            if (P.do_pick) warp_pick(P, nd, p, slot, lane);
        }
    }
}

// ---------------------------------------------------------------- block-per-node kernel (hubs)
__global__ void __launch_bounds__(HUB_THREADS) k_refresh_pick_hub(StepParams P) {
    __shared__ unsigned long long s_buf[CAND_CAP];
    __shared__ int s_count;
    __shared__ int s_done;
    if (__ldcg(P.status) != 0) return;
    const int lane = threadIdx.x & 31, wid = threadIdx.x >> 5;
    const int nwarps = HUB_THREADS / 32;
    const int nh = __ldcg(P.hub_count);
    const int W = P.W;
    for (int h = blockIdx.x; h < nh; h += gridDim.x) {
        const int p = __ldcg(P.hub_list + h);
        NodeCtx nd;
        load_node(P, p, nd, lane);
        int32_t* row = P.slots + (int64_t)nd.v * P.pitch;
        int32_t slot = -1;
        uint32_t evict = 0;
        if (wid == 0) {
            if (!P.init_rows && lane < W) slot = row[lane];
            evict = evict_mask_for(P, nd.v, lane);
        }
        const uint32_t nq = (nd.deg + 3u) >> 2;
        for (int attempt = (P.r < W ? 0 : 1); attempt < 3; ++attempt) {
            __syncthreads();
            if (threadIdx.x == 0) { s_count = 0; s_done = 0; }
            __syncthreads();
            uint32_t tinc = 0xFFFFFFFFu;
            if (attempt < 2) {
                tinc = threshold_for(attempt == 0 ? P.lambda_otf : P.lambda_full, nd.deg);
                // each warp scans a contiguous slice of quads into a private count, then appends
                const uint32_t per = (nq + nwarps - 1) / nwarps;
                const uint32_t qa = wid * per < nq ? wid * per : nq;
                const uint32_t qe = qa + per < nq ? qa + per : nq;
                const uint32_t lt = lanemask_lt();
                for (uint32_t qb = qa; qb < qe; qb += 32) {
                    const uint32_t q = qb + lane;
                    const uint4 o = philox4x32_10(q, (uint32_t)nd.v, P.step, P.word_fill, P.key0, P.key1);
                    const uint32_t kk[4] = {o.x, o.y, o.z, o.w};
#pragma unroll
                    for (int w = 0; w < 4; ++w) {
                        const uint32_t off = 4u * q + w;
                        const bool hit = (q < qe) && (off < nd.deg) && (kk[w] <= tinc);
                        const uint32_t b = __ballot_sync(FULL, hit);
                        if (b) {
                            int basepos = 0;
                            if (lane == 0) basepos = atomicAdd(&s_count, __popc(b));
                            basepos = __shfl_sync(FULL, basepos, 0);
                            if (hit) {
                                const int pos = basepos + __popc(b & lt);
                                if (pos < CAND_CAP) s_buf[pos] = ((unsigned long long)kk[w] << 32) | off;
                            }
                        }
                    }
                }
            } else if (wid == 0) {
                warp_exact_top(P, nd.v, nd.deg, s_buf, lane);
                if (lane == 0) s_count = W;
            }
            __syncthreads();
            if (wid == 0) {
                const bool ok = warp_refill(P, nd, s_buf, s_count, attempt == 2 || tinc == 0xFFFFFFFFu, evict, slot, lane);
                if (lane == 0) s_done = ok ? 1 : 0;
            }
            __syncthreads();
            if (s_done) break;
        }
        if (wid == 0) {
            if (P.init_rows) {
                if (lane < P.pitch) row[lane] = (lane < W) ? slot : -1;
            } else if ((evict >> lane) & 1u) {
                row[lane] = slot;
            }
            if (P.do_pick) warp_pick(P, nd, p, slot, lane);
        }
    }
}

cudaError_t launch_refresh_pick(const StepParams& p, int64_t n_bound, cudaStream_t s) {
    int64_t blocks = (n_bound + RP_WARPS - 1) / RP_WARPS;
    const int64_t cap = 148 * 8;
    if (blocks > cap) blocks = cap;
    if (blocks < 1) blocks = 1;
    k_refresh_pick<<<(int)blocks, RP_THREADS, 0, s>>>(p);
    int64_t hub_blocks = n_bound < 148 * 4 ? n_bound : 148 * 4;
    if (hub_blocks < 1) hub_blocks = 1;
    k_refresh_pick_hub<<<(int)hub_blocks, HUB_THREADS, 0, s>>>(p);
    count_launches(2);
    return cudaGetLastError();
}

}  // namespace gs
