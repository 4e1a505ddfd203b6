/* gso.h - CPU oracle for GraphSnapShot's cached multi-hop neighbour sampler.
 *
 * TEST INFRASTRUCTURE ONLY.  This is a plain, slow, single-threaded restatement of the
 * paper's sampler (static pre-sample, FCR / OTF refresh, shared-cache mode, sampling from
 * the cache hop by hop, relabel, block CSR, feature gather), used to check the CUDA library
 * and as the timed CPU baseline.  It shares no code with the CUDA path, and the product
 * never calls it.
 *
 * Method: paper Section "Algorithmic Design" - Algorithm 2 (OTF Refresh: Initialize,
 * RefreshCache, SampleBlocks) and Algorithm 3 (FCR: CacheRefresh, SampleBlocks); shared
 * cache per Section "Shared Cache Design".  All random choices come from one keyed
 * counter-based generator (Philox4x32-10, Salmon et al., SC'11) so results are unique.
 *
 * Pinned by tests against: Philox known-answer vectors, exact enumeration of the selection
 * law with injected keys, stationarity of uniform subsets under evict/refill, the BFS special
 * case, and the structural invariants of the method.
 * Parity unpinned: the paper's time / memory / accuracy tables (they need its datasets).
 *
 * Conventions
 *   - CSR row v lists the in-neighbours of v, ascending, no duplicates; indptr int64, ids int32.
 *   - fan-outs are listed input-layer-first; sampling step k = 0..L-1 starts at the seeds and
 *     uses layer l = L-1-k (SampleBlocks in Algorithms 2 and 3 walks the layers from the last down).
 *   - item order: a precedes b  <=>  (key32(a), a) < (key32(b), b).
 *   - key32(i) = word (i & 3) of Philox4x32-10(counter = (i >> 2, v, step, (purpose << 8) | tag),
 *     key = (seed low word, seed high word)); purpose 1 = FILL over edge offsets,
 *     2 = EVICT over slot indices, 3 = PICK over slot indices, 4 = FETCH over edge offsets;
 *     tag = layer, except FILL/EVICT in shared-cache mode which use 0xFF.
 */
#ifndef GSO_H
#define GSO_H
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

enum { GSO_MODE_FCR = 0, GSO_MODE_OTF = 1, GSO_MODE_FBL = 2, GSO_MODE_OTF_FETCH = 3 };
enum { GSO_FILL = 1, GSO_EVICT = 2, GSO_PICK = 3, GSO_FETCH = 4 };

typedef struct gso_sampler gso_sampler;

/* Replacement key function for tests that enumerate the selection law. */
typedef uint32_t (*gso_key_fn)(void* ctx, uint32_t purpose, uint32_t tag, uint32_t v, uint32_t step, uint32_t i);

void gso_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]);

/* r = number of slots refreshed per node: W for FCR, floor(gamma*W + 0.5) for OTF. */
int32_t gso_refresh_count(int mode, double gamma, int32_t W);

/* The graph arrays are borrowed (must outlive the sampler).  Returns NULL on bad arguments. */
gso_sampler* gso_create(int64_t num_nodes, const int64_t* indptr, const int32_t* indices,
                        int32_t num_hops, const int32_t* fanouts, int32_t cache_width,
                        uint64_t seed, int32_t shared);
void gso_destroy(gso_sampler*);
void gso_set_key_fn(gso_sampler*, gso_key_fn fn, void* ctx);
/* Dense/sparse split by degree threshold theta (paper Section "Graph Splitting and Sampling
 * Strategies"): nodes with degree <= theta are sampled by the FBL rule in every mode and never
 * touch the cache; theta < 0 switches the split off (the default). */
void gso_set_theta(gso_sampler*, int64_t theta);

/* Current cache row of node v (layer ignored in shared mode); untouched rows are the static
 * pre-sample.  out has cache_width entries, -1 = empty slot. */
int gso_cache_row(gso_sampler*, int32_t layer, int32_t v, int32_t* out);
/* Overwrite a cache row (used to resume from an exported cache). */
int gso_cache_set_row(gso_sampler*, int32_t layer, int32_t v, const int32_t* row);
/* One node's refresh (r slots) and pick at a given layer/step; exposed for sampled checks. */
int gso_refresh_node(gso_sampler*, int32_t layer, int32_t v, uint32_t step, int32_t r);
int gso_pick_node(gso_sampler*, int32_t layer, int32_t v, uint32_t step, int32_t* out, int32_t* count);
/* OTF Fetch pick of one node with n_fetch neighbours taken from the graph; cache not modified. */
int gso_fetch_node(gso_sampler*, int32_t layer, int32_t v, uint32_t step, int32_t n_fetch, int32_t* out,
                   int32_t* count);
/* Neighbours fetched from the graph per node in OTF Fetch: floor(delta*f + 0.5). */
int32_t gso_fetch_count(double delta, int32_t f);
/* Full Batch Load pick of one node (no cache involved); out has room for fanout entries. */
int gso_fbl_node(gso_sampler*, int32_t layer, int32_t v, uint32_t step, int32_t* out, int32_t* count);

/* Whole-cache refresh, the literal reading of Algorithms 2 and 3 (every T-th batch, all layers, all
 * rows): mode GSO_MODE_FCR replaces every row, GSO_MODE_OTF replaces refresh_count(gamma) slots of
 * every row, with the keys of `step` (>= 1).  Batches between two such refreshes sample with
 * GSO_MODE_OTF and gamma = 0 (SampleFromCache only). */
int gso_refresh_all(gso_sampler*, int mode, double gamma, uint32_t step);

/* One batch.  mode/gamma as in the paper (gamma ignored for FCR and FBL).  GSO_MODE_FBL samples
 * every hop straight from the graph and leaves the cache untouched; for GSO_MODE_OTF_FETCH
 * `gamma` carries the fetch rate delta, and the cache is not modified either.  step >= 1.  Seeds must be distinct.
 * Returns 0, or nonzero on bad arguments. Results stay valid until the next call. */
int gso_sample_batch(gso_sampler*, const int32_t* seeds, int32_t num_seeds, int mode, double gamma, uint32_t step);

int32_t gso_num_nodes(const gso_sampler*, int32_t k);          /* n_k, k = 0..L   */
int32_t gso_num_edges(const gso_sampler*, int32_t layer);      /* edges of block `layer` */
const int32_t* gso_frontier(const gso_sampler*);               /* n_L global ids; prefix n_k = frontier_k */
const int32_t* gso_block_indptr(const gso_sampler*, int32_t layer);   /* [num_dst+1] */
const int32_t* gso_block_indices(const gso_sampler*, int32_t layer);  /* local src ids */
const int32_t* gso_block_picked(const gso_sampler*, int32_t layer);   /* global src ids */
int64_t gso_stat_refreshed(const gso_sampler*);                /* nodes refreshed in the last batch */
int64_t gso_stat_scanned(const gso_sampler*);                  /* sum of their degrees */

/* out[p, :] = X[ids[p], :], rows of row_bytes bytes, strides in bytes. */
void gso_gather(const void* X, int64_t ld_bytes, int64_t row_bytes, const int32_t* ids, int64_t n,
                void* out, int64_t out_ld_bytes);

#ifdef __cplusplus
}
#endif
#endif
