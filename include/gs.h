/* gs.h - C ABI of the B200 cached neighbour sampler (GraphSnapShot's GraphSDSampler hot path).
 *
 * The library keeps a per-node cache of fixed-width neighbour slots next to a CSR graph, and
 * per mini-batch refreshes the cached rows of the frontier's nodes (all slots: Fully Cache
 * Refresh; a fraction gamma of them: On-The-Fly), samples each hop's fan-out from the cache,
 * relabels global ids to block-local ids, builds every hop's block CSR and gathers the input
 * nodes' feature rows.  Every step runs in CUDA kernels built for sm_100a; there is no CPU
 * fallback.
 *
 * General rules
 *   - Pointers named d_* are DEVICE pointers, h_* are HOST pointers.  All device buffers are
 *     owned by the caller and must outlive the handle that borrows them.  The library allocates
 *     no device memory; the two opaque handles are small host objects.
 *   - Every call returns a gs_status; nothing throws, traps or aborts.  Host-side checks fail
 *     before any kernel is launched.  Problems only the device can see (a seed id out of range,
 *     a duplicate seed) set a status word that gs_batch_counts / gs_sync_status return; the
 *     kernels of that batch then write nothing further.
 *   - All work is enqueued on `stream` (a cudaStream_t passed as void*, NULL = default stream)
 *     and is asynchronous unless a call says it synchronises.
 *     The kernels of a batch are launched with programmatic stream serialization (a kernel is set
 *     up on the GPU while its predecessor drains and waits for it before it reads anything); towards
 *     other work on `stream` the usual stream order holds.
 *   - Graph contract: CSR row v lists the in-neighbours of v in ascending order without
 *     duplicates; num_nodes < 2^31; indptr is int64, ids are int32.
 *   - Fan-outs are listed input-layer-first.  Sampling step k = 0..L-1 starts at the seeds and
 *     uses layer l = L-1-k (the layer loop of SampleBlocks in Algorithm 2 runs from the last layer down).
 *   - Randomness: every choice orders items by (key32(item), item) ascending where key32(i) is
 *     word (i & 3) of Philox4x32-10(counter = (i >> 2, node, step, (purpose << 8) | tag),
 *     key = (seed low word, seed high word)); purpose 1 = FILL over edge offsets of the node's
 *     CSR row, 2 = EVICT over slot indices, 3 = PICK over slot indices; tag = layer, except
 *     FILL/EVICT of a shared cache, which use 0xFF.  The result of a call is therefore unique.
 */
#ifndef GS_H
#define GS_H
#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef struct gs_graph gs_graph; /* opaque host object */
typedef struct gs_cache gs_cache; /* opaque host object */

typedef enum {
    GS_OK = 0,
    GS_ERR_ARG = 1,       /* NULL pointer, size or parameter out of its documented range */
    GS_ERR_ALIGN = 2,     /* a device pointer is not aligned as documented */
    GS_ERR_RANGE = 3,     /* device-detected: a seed id outside [0, num_nodes) */
    GS_ERR_WORKSPACE = 4, /* a caller-provided buffer is smaller than the *_bytes call reports */
    GS_ERR_DUP_SEED = 5,  /* device-detected: the same seed id twice in one batch */
    GS_ERR_CUDA = 6       /* a CUDA runtime call failed; see gs_last_error() */
} gs_status;

typedef enum { GS_MODE_FCR = 0, GS_MODE_OTF = 1, GS_MODE_FBL = 2, GS_MODE_OTF_FETCH = 3 } gs_mode;
typedef enum { GS_F32 = 0, GS_BF16 = 1 } gs_dtype;

#define GS_MAX_HOPS 8
#define GS_MAX_CACHE_WIDTH 32

/* Graph "on disk" in the paper's terms (Section "System Components": the full graph G=(V,E) and
 * the node embeddings H_v): a CSR adjacency and a row-major feature matrix, both resident in
 * device memory and borrowed.
 *   d_indptr   int64[num_nodes+1], 8-byte aligned     d_indices  int32[num_edges], 4-byte aligned
 *   d_features [num_nodes][feat_ld] elements of `dtype` (feat_ld >= feat_dim, in elements);
 *              may be NULL if gs_gather_features is never called.
 * Validates sizes and alignment on the host only; launches nothing. */
gs_status gs_graph_create(int64_t num_nodes, int64_t num_edges, const int64_t* d_indptr,
                          const int32_t* d_indices, const void* d_features, gs_dtype dtype,
                          int32_t feat_dim, int64_t feat_ld, gs_graph** out);
void gs_graph_destroy(gs_graph*);

/* How gs_gather_features copies the rows of this graph.  0 (the default) and -1: rows of 128 to 512 bytes that
 * are 64-byte aligned on both sides (base, pitch and row size) move as bulk copies staged through shared memory,
 * a persistent grid of a few blocks per SM - the fastest when the gather has the GPU to itself; other rows take
 * the load/store kernel (grid: 256 blocks per SM with 0; 16 with -1, which says that nothing runs beside the
 * gather).  A positive value asks for the load/store kernel with a grid of at most
 * (SM count) * blocks_per_sm blocks of 256 threads (8 are resident per SM): many short blocks (256 - 1024) let
 * kernels of a concurrent higher-priority stream start at once.
 * gs_gather_status synchronises `stream` and reports whether a bulk-copy gather ever gave up a (bounded) wait. */
gs_status gs_graph_set_gather_grid(gs_graph*, int32_t blocks_per_sm);
gs_status gs_gather_status(void* stream);

/* Optional one-pass check of the graph contract on the device: row offsets start at 0, end at
 * num_edges and never decrease; every neighbour id lies in [0, num_nodes); each row is strictly
 * ascending (sorted, no duplicate neighbour) - the sampler relies on all of it and does not
 * re-check it per batch.  Synchronises `stream`.  *h_first_bad_row = -1 and GS_OK if the graph
 * is valid, else the lowest offending row and GS_ERR_ARG.  Uses an 8-byte device variable of the
 * library: calls must not overlap. */
gs_status gs_graph_validate(const gs_graph*, void* stream, int64_t* h_first_bad_row);

/* Bytes of device memory the cache needs: a small state header, the relabel table (8 bytes per
 * node) and the slot rows (num_hops caches, or one if shared != 0). */
gs_status gs_cache_bytes(const gs_graph*, int32_t num_hops, int32_t cache_width, int32_t shared, size_t* bytes);

/* Bytes of device scratch one gs_sample_batch call with at most max_seeds seeds needs.  The
 * per-hop block arrays returned by gs_sample_batch live inside it. */
gs_status gs_workspace_bytes(const gs_graph*, int32_t num_hops, const int32_t* fanouts, int32_t max_seeds, size_t* bytes);

/* Static pre-sample (paper Algorithm 2, Initialize step; Section "Static and Dynamic
 * Sampling").  For every node and every layer (one row per node if shared):
 * degree <= cache_width -> the row is the adjacency in CSR order, remaining slots -1; otherwise
 * the row holds the cache_width neighbours first in FILL order at step 0, in that order.
 *   fanouts          h_ int32[num_hops], each in [1, cache_width]
 *   cache_width      in [1, GS_MAX_CACHE_WIDTH]
 *   d_cache_storage  256-byte aligned, cache_bytes >= gs_cache_bytes(...); owned by the caller,
 *                    initialised here, then read and written by every gs_sample_batch.
 * Enqueues the kernels on `stream`; does not synchronise. */
gs_status gs_cache_init(const gs_graph*, int32_t num_hops, const int32_t* fanouts, int32_t cache_width,
                        uint64_t seed, int32_t shared, void* d_cache_storage, size_t cache_bytes,
                        void* stream, gs_cache** out);
void gs_cache_destroy(gs_cache*);

/* Dense / sparse split (paper Section "Graph Splitting and Sampling Strategies": nodes with
 * degree > theta form the dense part, which is cached and refreshed by FCR / OTF; the remaining,
 * sparse part is loaded from the graph for every batch).  A split cache stores rows only for the
 * dense part, plus a 4-byte row index per node, instead of one row per node.
 *   theta        in [cache_width, 128]
 *   dense_rows   the number of nodes with degree > theta, counted by the caller (the storage is
 *                sized from it); gs_cache_init_split verifies it on the device and returns
 *                GS_ERR_ARG if it is wrong
 * Sampling with a split cache: a node of the sparse part is sampled by the Full Batch Load rule in
 * every mode (all neighbours if there are at most f_l, else the f_l edge offsets first in FETCH
 * order, emitted in ascending offset) and is never refreshed; the dense part behaves exactly as
 * with gs_cache_init.  gs_cache_read_rows returns -1 slots for sparse nodes.
 * gs_cache_init_split synchronises `stream` once (to verify dense_rows). */
gs_status gs_cache_bytes_split(const gs_graph*, int32_t num_hops, int32_t cache_width, int32_t shared,
                               int64_t dense_rows, size_t* bytes);
/* Counts the nodes with degree > theta on the device (the dense_rows argument above and below) and
 * synchronises `stream`.  Uses an 8-byte device variable of the library: calls must not overlap. */
gs_status gs_graph_count_dense(const gs_graph*, int32_t theta, void* stream, int64_t* h_dense_rows);
gs_status gs_cache_init_split(const gs_graph*, int32_t num_hops, const int32_t* fanouts, int32_t cache_width,
                              uint64_t seed, int32_t shared, int32_t theta, int64_t dense_rows,
                              void* d_cache_storage, size_t cache_bytes, void* stream, gs_cache** out);

/* Whole-cache refresh: the refresh exactly as Algorithms 2 and 3 write it (their periodic-refresh
 * condition on the batch counter t and the interval T: RefreshCache / CacheRefresh over all layers) - every cached row of every layer's cache, not only the
 * rows of a batch's frontier.  The caller owns the schedule: every T-th batch it calls this with
 * that batch's step, and samples all batches with gs_sample_batch(GS_MODE_OTF, gamma = 0), which is
 * SampleFromCache alone.
 *   mode   GS_MODE_FCR: all W slots of every row are replaced; GS_MODE_OTF: floor(gamma*W + 0.5)
 *          slots per row (Section "OTF Refresh"); other modes: GS_ERR_ARG
 *   step   >= 1; keys of (node, layer, step) as in gs_sample_batch, so refreshing a node here or
 *          through a batch of the same step gives the same row
 * Rows holding their whole adjacency (degree <= cache_width) and the sparse part of a split cache
 * are left alone.  Asynchronous on `stream`; needs no workspace (between batches the cache's own
 * relabel table is idle and serves as scratch).  Must not overlap a batch on the same cache, and
 * it clears the counts of the previous batch (gs_batch_counts, gs_batch_stats). */
gs_status gs_cache_refresh_all(gs_cache*, gs_mode mode, double gamma, uint32_t step, void* stream);

/* One hop's message-flow graph ("blocks" of Algorithm 2/3), stored destination-major.  The
 * destination nodes are the first *d_num_dst entries of the input-node list, the source nodes its
 * first *d_num_src entries (so sources begin with the destinations).  Counts are device scalars;
 * max_* are host-side upper bounds that size the arrays. */
typedef struct {
    int32_t max_dst, max_src, max_edges;
    const int32_t* d_num_dst;   /* device scalar */
    const int32_t* d_num_src;   /* device scalar */
    const int32_t* d_num_edges; /* device scalar */
    const int32_t* d_indptr;    /* [num_dst + 1] offsets into d_indices */
    const int32_t* d_indices;   /* [num_edges] block-local source ids */
} gs_block;

/* One mini-batch (paper Algorithm 2 RefreshCache + SampleBlocks for GS_MODE_OTF, Algorithm 3
 * CacheRefresh + SampleBlocks for GS_MODE_FCR; Section "Shared Cache Design" when the cache was
 * created shared).  For step k = 0..L-1 with layer l = L-1-k:
 *   refresh  every frontier node with degree > cache_width gets r of its slots replaced
 *            (r = cache_width for FCR, floor(gamma*cache_width + 0.5) for OTF): the r slot indices
 *            first in EVICT order are dropped, the others stay in place, and the dropped slots
 *            (ascending) receive the neighbours first in FILL order among those not retained.
 *            With a shared cache a node is refreshed only at the step it enters the frontier.
 *   pick     all cached neighbours if there are at most f_l, else the f_l slots first in PICK
 *            order, emitted in ascending slot index;
 *   relabel  next frontier = frontier followed by unseen picked ids in row-major order.
 * GS_MODE_FBL (the paper's Full Batch Load, Section "Full Batch Load (FBL)": no cache, every
 * neighbourhood is re-sampled from the graph) skips refresh and cache altogether: a node with at
 * most f_l neighbours takes them all, otherwise the f_l edge offsets first in FETCH order
 * (purpose 4, tag = layer, this step) are taken and emitted in ascending offset.  The cache is
 * neither read nor written; gamma is ignored.
 * GS_MODE_OTF_FETCH (the paper's second OTF mode, Section "OTF Fetch": the sample is
 * delta * FetchFromDisk + (1 - delta) * SampleFromCache) takes `gamma` as the fetch rate delta and
 * never modifies the cache.  A row that holds its whole adjacency is sampled as in `pick`.
 * Otherwise n = floor(delta*f_l + 0.5) neighbours are fetched from the graph and f_l - n come from
 * the cache: first the f_l - n slots first in PICK order (ascending slot index), then the n edge
 * offsets first in FETCH order among those whose neighbour is not one of these cache picks.
 * Arguments
 *   d_seeds      int32[num_seeds], distinct ids in [0, num_nodes); 1 <= num_seeds <= the
 *                max_seeds the workspace was sized for
 *   gamma        in [0, 1] (ignored for FCR);  step >= 1 (step 0 is the pre-sample)
 *   d_workspace  256-byte aligned, >= gs_workspace_bytes(..., num_seeds)
 *   blocks       h_ array of num_hops entries, filled by layer (blocks[0] = input side)
 *   d_input_nodes / d_num_input_nodes   receive device pointers to the global ids of the input
 *                nodes (the last frontier) and to their count
 * Block arrays and the input-node list stay valid until the next call on the same workspace.
 * Asynchronous.  Calls on one cache must not overlap on the device. */
gs_status gs_sample_batch(gs_cache*, const int32_t* d_seeds, int32_t num_seeds, gs_mode mode, double gamma,
                          uint32_t step, void* d_workspace, size_t workspace_bytes, void* stream,
                          gs_block* blocks, const int32_t** d_input_nodes, const int32_t** d_num_input_nodes);

/* Caller-owned output arrays of one hop for gs_sample_batch_noalloc (capacities in int32 entries). */
typedef struct {
    int32_t* d_indptr;
    int64_t indptr_capacity;
    int32_t* d_indices;
    int64_t indices_capacity;
} gs_block_buffers;

/* Bytes of the scratch array built into the library for gs_sample_batch_noalloc.  A GPU holds this
 * much device memory from the first gs_cache_init / gs_cache_init_split on it (which looks the
 * array up, the moment the CUDA runtime creates it there) until the process exits. */
#define GS_NOALLOC_SCRATCH_BYTES (64u << 20)

/* The same mini-batch as gs_sample_batch, for callers that cannot provide a scratch workspace
 * because they are not allowed to allocate device memory (a memory pool owns the whole device, a
 * host application hands out fixed buffers, a start-up memory budget is enforced).  The paper
 * has no counterpart to this call; it exists only for such deployments.  It allocates nothing
 * (no cudaMalloc / cudaFree, no allocating library routine): the scratch is a fixed array of
 * GS_NOALLOC_SCRATCH_BYTES inside the library, and the results go to buffers the caller passes:
 *   d_input_nodes   int32[input_nodes_capacity] receives the input-node list (the last frontier);
 *                   4-byte aligned
 *   h_buffers       h_ array of num_hops entries, by layer: where each block's offsets and
 *                   block-local source ids go.  With n_0 = num_seeds, m_k = n_k * fanout of step k
 *                   and n_{k+1} = min(num_nodes, n_k + m_k), the block of step k needs n_k + 1
 *                   offsets and m_k indices, and the input-node list needs n_L ids.
 *                   d_indptr must be 4-byte aligned and d_indices 16-BYTE aligned (the ids are
 *                   stored four at a time); a caller that carves its arrays out of one buffer
 *                   rounds each d_indices start up to 16 bytes.  GS_ERR_ALIGN otherwise.
 *   blocks          filled as by gs_sample_batch, pointing into the caller's buffers
 *   d_num_input_nodes  receives a device pointer to the count (may be NULL)
 * Everything else (seeds, mode, gamma, step, results, status reporting through gs_batch_counts) is
 * as for gs_sample_batch, and the results are bit-identical.
 * Limits and rules
 *   - A batch needs as much scratch as gs_workspace_bytes reports for it; if that exceeds
 *     GS_NOALLOC_SCRATCH_BYTES the call returns GS_ERR_WORKSPACE (message with both sizes) and
 *     launches nothing.  Too-small output buffers are rejected the same way, misaligned ones with
 *     GS_ERR_ALIGN; every check runs on the host before the first launch.
 *   - The device address of the built-in array is looked up once per device, with that device
 *     current: by gs_cache_init / gs_cache_init_split, which is also when the array starts to
 *     occupy memory there, so a deployment sees the full footprint at set-up.  Should the first
 *     use on a device be this call itself (a cache created while another device was current), the
 *     lookup happens here: make that first call outside any stream capture.
 *   - All calls on a device share the one array and it keeps the previous call's contents; the
 *     kernels initialise every part of it they read, so nothing has to be cleared between calls.
 *     Two calls whose kernels overlap on the GPU (different streams, different caches) race on
 *     the array: run them one after the other. */
gs_status gs_sample_batch_noalloc(gs_cache*, const int32_t* d_seeds, int32_t num_seeds, gs_mode mode, double gamma,
                                  uint32_t step, int32_t* d_input_nodes, int64_t input_nodes_capacity,
                                  const gs_block_buffers* h_buffers, void* stream, gs_block* blocks,
                                  const int32_t** d_num_input_nodes);

/* Same batch for a caller whose seeds are in HOST memory: copies h_seeds to the device, runs the
 * batch, copies the counts back and synchronises `stream`.
 *   h_num_nodes  int32[num_hops + 1]: n_0 (seeds) .. n_L (input nodes), by sampling step
 *   h_num_edges  int32[num_hops]: edges per block, by layer
 * Returns the device status of the batch. */
gs_status gs_sample_batch_host(gs_cache*, const int32_t* h_seeds, int32_t num_seeds, gs_mode mode, double gamma,
                               uint32_t step, void* d_workspace, size_t workspace_bytes, void* stream,
                               gs_block* blocks, const int32_t** d_input_nodes,
                               int32_t* h_num_nodes, int32_t* h_num_edges);

/* Synchronises `stream` and returns the counts of the last batch on this cache (layout as in
 * gs_sample_batch_host; either pointer may be NULL) and its device status. */
gs_status gs_batch_counts(gs_cache*, void* stream, int32_t* h_num_nodes, int32_t* h_num_edges);

/* Feature gather (the paper's "load embeddings", Section "System Components"):
 * out[p, :] = features[ids[p], :] for p < count, a bitwise copy.
 *   d_ids            int32 ids in [0, num_nodes); any other id is skipped (its output row is left as it is)
 *   d_count_or_null  device scalar with the row count, or NULL to use count_bound
 *   count_bound      rows d_out has room for (and the count, when d_count_or_null is NULL)
 *   d_out            [count_bound][out_ld] elements of the graph's dtype, out_ld >= feat_dim
 * Uses 16-byte accesses when base pointers and both row pitches allow it, narrower otherwise. */
gs_status gs_gather_features(const gs_graph*, const int32_t* d_ids, const int32_t* d_count_or_null,
                             int32_t count_bound, void* d_out, int64_t out_ld, void* stream);

/* out[i, :] = src[ids[i] - first_row, :] for any row-major matrix on the device (the copy kernel
 * of gs_gather_features).  `src` holds the src_rows rows first_row, first_row + 1, ... of a larger
 * matrix - a feature shard - and ids are global; an id outside [first_row, first_row + src_rows)
 * is skipped (its output row is left as it is).  row_elems, src_ld, out_ld in elements of `dtype`. */
gs_status gs_gather_rows(const void* d_src, gs_dtype dtype, int32_t row_elems, int64_t src_ld, int64_t first_row,
                         int64_t src_rows, const int32_t* d_ids, const int32_t* d_count_or_null, int32_t count_bound, void* d_out,
                         int64_t out_ld, void* stream);

/* The feature step of a sharded run as ONE kernel over peer memory: out[i, :] = row ids[i] of a
 * matrix whose rows are split over `world` shards of S = ceil(num_rows / world) rows; shard o holds
 * rows [o*S, (o+1)*S) and starts at h_shard_bases[o] (a HOST array of DEVICE addresses - this
 * GPU's own memory or peer GPUs' memory mapped into this process, e.g. CUDA IPC or a symmetric
 * allocation; mapping is the caller's).  Each row is read with plain 16-byte streaming loads
 * straight from its owner and written to `d_out`: the row crosses NVLink once, no staging buffer,
 * no exchange of ids.  ids outside [0, num_rows) are skipped.  All shards share src_ld. */
gs_status gs_gather_rows_peer(const void* const* h_shard_bases, int32_t world, int64_t num_rows, gs_dtype dtype,
                              int32_t row_elems, int64_t src_ld, const int32_t* d_ids, const int32_t* d_count_or_null,
                              int32_t count_bound, void* d_out, int64_t out_ld, void* stream);

/* ---- Node-sharded sampling over several GPUs (the paper's Section "Shared Cache Mode" speaks of a
 * cache shared by several trainer processes; the partition and the exchange are this
 * library's).  Nodes are partitioned by id range: shard o of `world` owns the nodes
 * [o*S, (o+1)*S), S = ceil(num_nodes / world), with their CSR rows, cache rows and feature rows.
 * A shard's gs_graph has the full num_nodes and an indptr in which only the owned rows are
 * non-empty; its cache is created with gs_cache_init_split, so only owned dense rows use memory.
 * One hop (sampling step k, layer L-1-k) of a rank's batch:
 *   1. gs_shard_bucket           frontier_k grouped by owner            (requester)
 *   2. exchange the groups (all-to-all; the caller's, e.g. NCCL)
 *   3. gs_shard_sample_rows      refresh + pick for each received list  (owner)
 *   4. exchange the rows of picks back
 *   5. gs_shard_extend           dedup + relabel + block CSR            (requester)
 * and after the last hop the same exchange with gs_gather_rows for the feature rows.  Every
 * random choice is keyed by (seed, node, item, step), so the rows an owner returns are the rows
 * a single device would compute, and refreshing a node twice in one step (two ranks ask for it)
 * gives the same row as once.  A sharded run therefore equals one sampler, with dense/sparse
 * split theta, that takes the ranks' batches of a step one after the other.  All ranks use the
 * same step for the batches they run together. */

/* Groups n node ids by owner.  d_sorted[n]: the ids, owner 0's first (order inside a group is
 * unspecified); d_slot[n]: position of d_nodes[i] in d_sorted; d_counts: int32[2*world + 1], on
 * return words [0, world) hold the group sizes and word 2*world is 0 or GS_ERR_RANGE (an id outside
 * [0, num_nodes)); the words between are scratch.  world <= 64.  Asynchronous on `stream`. */
gs_status gs_shard_bucket(const int32_t* d_nodes, int32_t n, int64_t num_nodes, int32_t world, int32_t* d_sorted,
                          int32_t* d_slot, int32_t* d_counts, void* stream);
/* The same for a list whose length is a device scalar (the frontier of the previous hop: *d_n, e.g.
 * gs_block.d_num_src), of at most n_bound ids: the requester needs no host copy of the frontier's size
 * before it buckets; the group sizes it reads back for the exchange add up to the length.  *d_n > n_bound
 * sets word 2*world to GS_ERR_WORKSPACE (only the first n_bound ids are grouped). */
gs_status gs_shard_bucket_counted(const int32_t* d_nodes, const int32_t* d_n, int32_t n_bound, int64_t num_nodes,
                                  int32_t world, int32_t* d_sorted, int32_t* d_slot, int32_t* d_counts, void* stream);

/* The same with every owner's group at a fixed pitch: owner o's ids are d_sorted[o*capacity ..
 * o*capacity + counts[o]) (d_sorted holds world*capacity ids, the rest of a segment is left as it is), so the
 * groups can be exchanged in equal splits without the host ever reading a size; the counts travel as a
 * device array beside them.  d_n_or_null as for gs_shard_bucket_counted (NULL: all n_bound ids).  A group
 * larger than `capacity` sets word 2*world to GS_ERR_WORKSPACE; its surplus nodes get slot -1 and are dropped
 * (gs_shard_extend_fixed then reports them too). */
gs_status gs_shard_bucket_fixed(const int32_t* d_nodes, const int32_t* d_n_or_null, int32_t n_bound, int64_t num_nodes,
                                int32_t world, int32_t capacity, int32_t* d_sorted, int32_t* d_slot, int32_t* d_counts,
                                void* stream);

/* Owner side.  For n distinct nodes of this shard: refresh (per mode / rate, exactly as
 * gs_sample_batch does for a frontier at `layer`) and pick; d_picks[n][fanout(layer)] receives the
 * picks of node i in the order a local batch would emit them, padded with -1.  Works on state of
 * its own (a second header) and does not touch the relabel table, so it may run between the hops
 * of this rank's own batch.  Lists of different requesters go in separate calls (a node may
 * appear in several of them).  Workspace: gs_shard_workspace_bytes(graph, fanout(layer), n).
 * gs_shard_sample_rows_counted takes the list's length from the device (*d_n, at most n_bound; e.g. a word of
 * the exchanged counts of gs_shard_bucket_fixed) and writes only that many rows of d_picks[n_bound][fanout].
 * gs_shard_status synchronises `stream`, reports a bad node id met by any list served since its last call
 * (after such an id the later lists are not served) and clears that state. */
gs_status gs_shard_workspace_bytes(const gs_graph*, int32_t fanout, int32_t max_nodes, size_t* bytes);
gs_status gs_shard_sample_rows(gs_cache*, const int32_t* d_nodes, int32_t n, int32_t layer, gs_mode mode, double rate,
                               uint32_t step, void* d_workspace, size_t workspace_bytes, void* stream, int32_t* d_picks);
gs_status gs_shard_sample_rows_counted(gs_cache*, const int32_t* d_nodes, const int32_t* d_n, int32_t n_bound, int32_t layer,
                                       gs_mode mode, double rate, uint32_t step, void* d_workspace, size_t workspace_bytes,
                                       void* stream, int32_t* d_picks);
gs_status gs_shard_status(gs_cache*, void* stream);

/* Owner side, all requesters' fixed-pitch lists at once (d_lists[world][capacity], lengths d_counts[world], as
 * they arrive from the exchange): a node that several requesters ask for - every hub - is sampled once.
 * gs_shard_merge gives every requested node one place in d_distinct (at most min(world*capacity, rows_owned)
 * ids, in no particular order); d_num_distinct: int32[2] on the device, [0] = how many, [1] = 0 or GS_ERR_RANGE
 * (an id outside the rows this shard owns, [first_row, first_row + rows_owned); such entries are skipped).
 * d_index: int32[rows_owned], owned by the caller, all -1 before the first call; it holds the nodes' places
 * until gs_shard_fan_out has run.  Then gs_shard_sample_rows_counted(d_distinct, d_num_distinct, ...) samples the
 * distinct nodes into d_rows[..][fanout], and gs_shard_fan_out copies every list entry's row to
 * d_out[world*capacity][fanout] (the reply at the lists' pitch) and puts d_index back to all -1.  The rows are
 * the ones the per-list calls give: picks are keyed by (node, step), not by who asks. */
gs_status gs_shard_merge(const int32_t* d_lists, const int32_t* d_counts, int32_t world, int32_t capacity, int64_t first_row,
                         int64_t rows_owned, int32_t* d_index, int32_t* d_distinct, int32_t* d_num_distinct, void* stream);
gs_status gs_shard_fan_out(const int32_t* d_lists, const int32_t* d_counts, int32_t world, int32_t capacity, int64_t first_row,
                           int64_t rows_owned, int32_t* d_index, const int32_t* d_distinct, const int32_t* d_num_distinct,
                           const int32_t* d_rows, int32_t fanout, int32_t* d_out, void* stream);

/* Requester side, hop k = 0 .. num_hops-1 in order.  d_reply[n_k][fanout(L-1-k)]: the owners' rows
 * in d_sorted order; d_slot[n_k] as returned by gs_shard_bucket for frontier_k.  k = 0 starts a new
 * batch and takes the seeds (distinct, as for gs_sample_batch); later hops ignore d_seeds and
 * num_seeds.  The workspace is the one of gs_sample_batch (gs_workspace_bytes for num_seeds) and
 * must stay untouched between the hops of a batch.  A slot outside [0, n_k) or a pick outside
 * [0, num_nodes) sets the device status GS_ERR_RANGE (see gs_batch_counts).  Fills *block like gs_sample_batch fills
 * blocks[L-1-k]; *d_frontier is the frontier array (frontier_{k+1} is its prefix of
 * *block->d_num_src ids).  Counts: gs_batch_counts, as after gs_sample_batch. */
gs_status gs_shard_extend(gs_cache*, int32_t k, const int32_t* d_seeds, int32_t num_seeds, const int32_t* d_reply,
                          const int32_t* d_slot, void* d_workspace, size_t workspace_bytes, void* stream, gs_block* block,
                          const int32_t** d_frontier);
/* The same for replies at a fixed pitch (gs_shard_bucket_fixed): d_reply[reply_rows][fanout] with
 * reply_rows = world * capacity, d_slot the positions that call returned (required).  A slot outside
 * [0, reply_rows) sets GS_ERR_RANGE. */
gs_status gs_shard_extend_fixed(gs_cache*, int32_t k, const int32_t* d_seeds, int32_t num_seeds, const int32_t* d_reply,
                                int32_t reply_rows, const int32_t* d_slot, void* d_workspace, size_t workspace_bytes,
                                void* stream, gs_block* block, const int32_t** d_frontier);

/* Copy n logical cache rows (cache_width slots each, -1 = empty) of `layer` into d_out[n][cache_width]. */
gs_status gs_cache_read_rows(const gs_cache*, int32_t layer, const int32_t* d_nodes, int32_t n,
                             int32_t* d_out, void* stream);

/* Checkpoint / resume: the slot rows as one opaque blob of gs_cache_export_bytes bytes. */
gs_status gs_cache_export_bytes(const gs_cache*, size_t* bytes);
gs_status gs_cache_export(const gs_cache*, void* d_dst, size_t bytes, void* stream);
gs_status gs_cache_import(gs_cache*, const void* d_src, size_t bytes, void* stream);

/* Synchronises `stream` and copies four counters of the last batch into h_stats[4]:
 * [0] nodes whose refill had to be redone by a full rescan on one warp, [1] nodes handed to the
 * chunked multi-warp rescan, and, for a partial refresh (0 < r < cache_width) only,
 * [2] nodes refreshed, [3] Philox blocks (4 edge offsets each) the threshold scan evaluates.
 * Diagnostics only. */
gs_status gs_batch_stats(gs_cache*, void* stream, int64_t* h_stats);

/* Index (in int32 words from the start of the cache storage) of the four gs_batch_stats counters,
 * for callers that copy the state header asynchronously instead of synchronising per batch. */
int32_t gs_stats_word_offset(void);

/* Optional device-side timing of the kernels of gs_sample_batch.  Between _begin and _end every
 * batch (up to max_batches, in [1, 4096]) records CUDA events on its own stream around four
 * kernel groups of each sampling step: row counts / block offsets, threshold scan, finish (or
 * the fused refresh + pick kernels), dedup + relabel.  _end synchronises `stream`, writes the
 * summed milliseconds of the four groups to h_ms[4] and the number of batches timed to
 * *h_batches, and releases the events.  Events are host objects; no device memory is used. */
gs_status gs_cache_profile_begin(gs_cache*, int32_t max_batches);
gs_status gs_cache_profile_end(gs_cache*, void* stream, double* h_ms, int64_t* h_batches);

/* Synchronises `stream` and returns the device status of the last batch. */
gs_status gs_sync_status(gs_cache*, void* stream);

/* Selection tuning (never changes results, only which internal path finds them):
 * expected number of candidate edges kept by the threshold scan for an OTF refill and for a full
 * refill, and the degree above which a whole thread block scans one node.  Values <= 0 keep the
 * defaults. */
gs_status gs_cache_set_tuning(gs_cache*, double lambda_otf, double lambda_full, int32_t hub_degree);

/* How gs_sample_batch finds each id's first occurrence for the dedup + relabel of a step (the paper's
 * Algorithms 2 and 3 only say that the sampled neighbours become the next frontier and that blocks are
 * returned; the three methods give identical blocks and differ in speed only):
 *   GS_DEDUP_DIRECT            direct-address table of 8 bytes per graph node inside the cache storage;
 *                              every pick claims its position with one atomicMin.
 *   GS_DEDUP_HASH              open-addressing hash table of 1.5 x (frontier + picks) entries, rebuilt at
 *                              every sampling step inside the workspace: follows the batch, not the graph.
 *   GS_DEDUP_SORT              stable radix sort of (id, position) pairs; run heads are first occurrences.
 *   GS_DEDUP_AUTO (default)    per sampling step, by measurement on B200: the hash table when the direct
 *                              table is larger than 64 MiB (it then falls out of L2) and the step can hold
 *                              half a million keys or more, the direct table otherwise.
 * Applies to the following gs_sample_batch / gs_sample_batch_host / gs_sample_batch_noalloc calls on this
 * cache; the node-sharded calls always use the direct table. */
#define GS_DEDUP_DIRECT 0
#define GS_DEDUP_HASH 1
#define GS_DEDUP_SORT 2
#define GS_DEDUP_AUTO 3
gs_status gs_cache_set_dedup(gs_cache*, int32_t method);

/* Test knob, process-wide: no kernel of the library is launched with more than max_blocks thread
 * blocks (0 restores the designed grids).  Every kernel walks its work with a grid-stride or
 * work-counter loop, so results never depend on the grid; tests use caps of 1-3 blocks to make
 * each block walk many tiles, a path the designed grids only take on the largest batches. */
gs_status gs_debug_set_grid_cap(int32_t max_blocks);

/* Measured integer-arithmetic ceilings of the current device, for reporting the threshold scan
 * against its roofline (the key function of every selection is Philox4x32-10, Salmon et al. SC'11;
 * the scan evaluates one block per four edge offsets and is bound by this arithmetic, not by memory).
 * Runs a kernel that does nothing but the chosen arithmetic for about `milliseconds` (1..2000) on
 * `stream`, synchronises, and returns the sustained rate in *h_units_per_second:
 *   what = 0  Philox4x32-10 blocks with the scan's threshold test (four blocks per thread in flight)
 *   what = 1  32x32->64-bit multiplies (a Philox block has 20)
 *   what = 2  three-input logic operations (a Philox block has 20)
 * Uses CUDA events (host objects) and a 4-byte device variable of the library; allocates nothing. */
gs_status gs_alu_ceiling(int32_t what, int32_t milliseconds, void* stream, double* h_units_per_second);

/* Number of kernels this library has launched in the calling process (monotonic). */
int64_t gs_kernel_launches(void);

/* Message of the last failing call in this thread ("" if none). */
const char* gs_last_error(void);

#ifdef __cplusplus
}
#endif
#endif
