/* gso.c - CPU oracle (test infrastructure; see gso.h).  Plain C, single thread, no blocking,
 * no fusion: every selection is "sort all items by (key, index), take a prefix". */
#include "gso.h"

#include <math.h>
#include <stdlib.h>
#include <string.h>

#define GSO_MAX_HOPS 8

struct gso_sampler {
    int64_t N;
    const int64_t* indptr;
    const int32_t* indices;
    int32_t L, W, shared;
    int64_t theta;   /* dense/sparse split: rows with degree <= theta are never cached (-1: no split) */
    int32_t fanouts[GSO_MAX_HOPS];
    uint64_t seed;
    gso_key_fn key_fn;
    void* key_ctx;
    int32_t num_caches;
    int32_t** rows[GSO_MAX_HOPS]; /* rows[c][v] = NULL (untouched) or W slots */
    /* last batch */
    int32_t* frontier;
    int64_t frontier_cap;
    int32_t n[GSO_MAX_HOPS + 1];
    int32_t m[GSO_MAX_HOPS];
    int32_t* blk_indptr[GSO_MAX_HOPS];
    int32_t* blk_indices[GSO_MAX_HOPS];
    int32_t* blk_picked[GSO_MAX_HOPS];
    int32_t* pos; /* N entries, -1 = not in the frontier */
    int64_t stat_refreshed, stat_scanned;
};

/* ------------------------------------------------------------------ Philox4x32-10 */
/* Salmon, Moraes, Dror, Shaw: "Parallel random numbers: as easy as 1, 2, 3" (SC'11). */
void gso_philox4x32_10(const uint32_t ctr[4], const uint32_t key[2], uint32_t out[4]) {
    uint32_t c0 = ctr[0], c1 = ctr[1], c2 = ctr[2], c3 = ctr[3];
    uint32_t k0 = key[0], k1 = key[1];
    for (int round = 0; round < 10; ++round) {
        uint64_t p0 = (uint64_t)0xD2511F53u * c0;
        uint64_t p1 = (uint64_t)0xCD9E8D57u * c2;
        uint32_t hi0 = (uint32_t)(p0 >> 32), lo0 = (uint32_t)p0;
        uint32_t hi1 = (uint32_t)(p1 >> 32), lo1 = (uint32_t)p1;
        uint32_t n0 = hi1 ^ c1 ^ k0;
        uint32_t n2 = hi0 ^ c3 ^ k1;
        c0 = n0; c1 = lo1; c2 = n2; c3 = lo0;
        k0 += 0x9E3779B9u;
        k1 += 0xBB67AE85u;
    }
    out[0] = c0; out[1] = c1; out[2] = c2; out[3] = c3;
}

static uint32_t key32(const gso_sampler* s, uint32_t purpose, uint32_t tag, uint32_t v, uint32_t step, uint32_t i) {
    if (s->key_fn) return s->key_fn(s->key_ctx, purpose, tag, v, step, i);
    uint32_t ctr[4] = { i >> 2, v, step, (purpose << 8) | tag };
    uint32_t key[2] = { (uint32_t)(s->seed & 0xFFFFFFFFu), (uint32_t)(s->seed >> 32) };
    uint32_t out[4];
    gso_philox4x32_10(ctr, key, out);
    return out[i & 3];
}

/* ------------------------------------------------------------------ ordering */
typedef struct { uint32_t key, idx; } item_t;

static int item_cmp(const void* a, const void* b) {
    const item_t* x = (const item_t*)a;
    const item_t* y = (const item_t*)b;
    if (x->key != y->key) return x->key < y->key ? -1 : 1;
    if (x->idx != y->idx) return x->idx < y->idx ? -1 : 1;
    return 0;
}

static int i32_cmp(const void* a, const void* b) {
    int32_t x = *(const int32_t*)a, y = *(const int32_t*)b;
    return x < y ? -1 : (x > y ? 1 : 0);
}

/* Sort `count` items (idx already set) by (key, idx). */
static void order_items(const gso_sampler* s, item_t* it, int64_t count, uint32_t purpose, uint32_t tag,
                        uint32_t v, uint32_t step) {
    for (int64_t t = 0; t < count; ++t) it[t].key = key32(s, purpose, tag, v, step, it[t].idx);
    qsort(it, (size_t)count, sizeof(item_t), item_cmp);
}

/* ------------------------------------------------------------------ helpers */
int32_t gso_refresh_count(int mode, double gamma, int32_t W) {
    if (mode == GSO_MODE_FCR) return W;
    double r = floor(gamma * (double)W + 0.5);
    if (r < 0) r = 0;
    if (r > W) r = W;
    return (int32_t)r;
}

int32_t gso_fetch_count(double delta, int32_t f) {
    double n = floor(delta * (double)f + 0.5);
    if (n < 0) n = 0;
    if (n > f) n = f;
    return (int32_t)n;
}

static int64_t degree(const gso_sampler* s, int32_t v) { return s->indptr[v + 1] - s->indptr[v]; }
static int32_t nbr(const gso_sampler* s, int32_t v, uint32_t i) { return s->indices[s->indptr[v] + (int64_t)i]; }
static int32_t cache_of(const gso_sampler* s, int32_t layer) { return s->shared ? 0 : layer; }
static uint32_t cache_tag(const gso_sampler* s, int32_t layer) { return s->shared ? 0xFFu : (uint32_t)layer; }

/* Static pre-sample of one row (Algorithm 2, Initialize): all neighbours if they fit, else the W
 * edge offsets first in FILL order at step 0, stored in that order. */
static void presample_row(const gso_sampler* s, int32_t layer, int32_t v, int32_t* row) {
    int64_t deg = degree(s, v);
    int32_t W = s->W;
    for (int32_t j = 0; j < W; ++j) row[j] = -1;
    if (deg <= W) {
        for (int64_t j = 0; j < deg; ++j) row[j] = nbr(s, v, (uint32_t)j);
        return;
    }
    item_t* it = (item_t*)malloc((size_t)deg * sizeof(item_t));
    for (int64_t i = 0; i < deg; ++i) it[i].idx = (uint32_t)i;
    order_items(s, it, deg, GSO_FILL, cache_tag(s, layer), (uint32_t)v, 0u);
    for (int32_t j = 0; j < W; ++j) row[j] = nbr(s, v, it[j].idx);
    free(it);
}

static int32_t* row_of(gso_sampler* s, int32_t layer, int32_t v) {
    int32_t c = cache_of(s, layer);
    int32_t* row = s->rows[c][v];
    if (!row) {
        row = (int32_t*)malloc((size_t)s->W * sizeof(int32_t));
        presample_row(s, layer, v, row);
        s->rows[c][v] = row;
    }
    return row;
}

/* Refresh r slots of v's row (Algorithm 2, RefreshCache; r = W is Algorithm 3's CacheRefresh):
 * the r slot indices first in EVICT order are dropped, the rest stay in place; the candidates
 * are the edge offsets whose neighbour is not retained, in FILL order at this step; the t-th
 * candidate goes into the t-th evicted slot, evicted slots taken in ascending slot index. */
static void refresh_row(gso_sampler* s, int32_t layer, int32_t v, uint32_t step, int32_t r) {
    int64_t deg = degree(s, v);
    int32_t W = s->W;
    if (deg <= W || r <= 0) return;
    if (r > W) r = W;
    int32_t* row = row_of(s, layer, v);
    uint32_t tag = cache_tag(s, layer);

    item_t slots[64];
    for (int32_t j = 0; j < W; ++j) slots[j].idx = (uint32_t)j;
    order_items(s, slots, W, GSO_EVICT, tag, (uint32_t)v, step);
    int evicted[64];
    memset(evicted, 0, sizeof(evicted));
    for (int32_t t = 0; t < r; ++t) evicted[slots[t].idx] = 1;

    item_t* cand = (item_t*)malloc((size_t)deg * sizeof(item_t));
    int64_t nc = 0;
    for (int64_t i = 0; i < deg; ++i) {
        int32_t u = nbr(s, v, (uint32_t)i);
        int retained = 0;
        for (int32_t j = 0; j < W; ++j)
            if (!evicted[j] && row[j] == u) retained = 1;
        if (!retained) cand[nc++].idx = (uint32_t)i;
    }
    order_items(s, cand, nc, GSO_FILL, tag, (uint32_t)v, step);
    int64_t t = 0;
    for (int32_t j = 0; j < W; ++j)
        if (evicted[j]) row[j] = nbr(s, v, cand[t++].idx);
    free(cand);
    s->stat_refreshed += 1;
    s->stat_scanned += deg;
}

/* SampleFromCache for one node: all cached neighbours if there are at most f, else the f slot
 * indices first in PICK order, emitted in ascending slot index. */
static int32_t pick_row(gso_sampler* s, int32_t layer, int32_t v, uint32_t step, int32_t* out) {
    int64_t deg = degree(s, v);
    int32_t W = s->W, f = s->fanouts[layer];
    int32_t c = (int32_t)(deg < W ? deg : W);
    const int32_t* row = row_of(s, layer, v);
    if (c <= f) {
        for (int32_t j = 0; j < c; ++j) out[j] = row[j];
        return c;
    }
    item_t slots[64];
    for (int32_t j = 0; j < c; ++j) slots[j].idx = (uint32_t)j;
    order_items(s, slots, c, GSO_PICK, (uint32_t)layer, (uint32_t)v, step);
    int32_t chosen[64];
    for (int32_t t = 0; t < f; ++t) chosen[t] = (int32_t)slots[t].idx;
    qsort(chosen, (size_t)f, sizeof(int32_t), i32_cmp);
    for (int32_t t = 0; t < f; ++t) out[t] = row[chosen[t]];
    return f;
}

/* Full Batch Load for one node (paper Section "Full Batch Load (FBL)": the neighbourhood is
 * re-sampled from the graph for every batch, no cache): all neighbours if there are at most f,
 * else the f edge offsets first in FETCH order at this step, emitted in ascending offset. */
static int32_t fbl_row(gso_sampler* s, int32_t layer, int32_t v, uint32_t step, int32_t* out) {
    int64_t deg = degree(s, v);
    int32_t f = s->fanouts[layer];
    if (deg <= f) {
        for (int64_t j = 0; j < deg; ++j) out[j] = nbr(s, v, (uint32_t)j);
        return (int32_t)deg;
    }
    item_t* it = (item_t*)malloc((size_t)deg * sizeof(item_t));
    for (int64_t i = 0; i < deg; ++i) it[i].idx = (uint32_t)i;
    order_items(s, it, deg, GSO_FETCH, (uint32_t)layer, (uint32_t)v, step);
    int32_t chosen[64];
    for (int32_t t = 0; t < f; ++t) chosen[t] = (int32_t)it[t].idx;
    free(it);
    qsort(chosen, (size_t)f, sizeof(int32_t), i32_cmp);
    for (int32_t t = 0; t < f; ++t) out[t] = nbr(s, v, (uint32_t)chosen[t]);
    return f;
}

/* OTF Fetch for one node (paper Section "OTF Fetch": the sample is part cache, part graph, with
 * fetch rate delta; the cache is not modified).  A row that holds its whole adjacency is sampled
 * like any cached row.  Otherwise n_fetch = floor(delta*f + 0.5) neighbours come from the graph and
 * f - n_fetch from the cache: the cache part is the f - n_fetch slots first in PICK order, emitted
 * in ascending slot index; the fetched part is the n_fetch edge offsets first in FETCH order among
 * those whose neighbour is not one of the cache picks, emitted in that order after the cache part. */
static int32_t fetch_row(gso_sampler* s, int32_t layer, int32_t v, uint32_t step, int32_t n_fetch, int32_t* out) {
    int64_t deg = degree(s, v);
    int32_t W = s->W, f = s->fanouts[layer];
    if (deg <= W || n_fetch <= 0) return pick_row(s, layer, v, step, out);
    if (n_fetch > f) n_fetch = f;
    int32_t n_cache = f - n_fetch;
    const int32_t* row = row_of(s, layer, v);
    item_t slots[64];
    for (int32_t j = 0; j < W; ++j) slots[j].idx = (uint32_t)j;
    order_items(s, slots, W, GSO_PICK, (uint32_t)layer, (uint32_t)v, step);
    int32_t chosen[64];
    for (int32_t t = 0; t < n_cache; ++t) chosen[t] = (int32_t)slots[t].idx;
    qsort(chosen, (size_t)n_cache, sizeof(int32_t), i32_cmp);
    for (int32_t t = 0; t < n_cache; ++t) out[t] = row[chosen[t]];
    item_t* cand = (item_t*)malloc((size_t)deg * sizeof(item_t));
    int64_t nc = 0;
    for (int64_t i = 0; i < deg; ++i) {
        int32_t u = nbr(s, v, (uint32_t)i);
        int taken = 0;
        for (int32_t t = 0; t < n_cache; ++t)
            if (out[t] == u) taken = 1;
        if (!taken) cand[nc++].idx = (uint32_t)i;
    }
    order_items(s, cand, nc, GSO_FETCH, (uint32_t)layer, (uint32_t)v, step);
    for (int32_t t = 0; t < n_fetch; ++t) out[n_cache + t] = nbr(s, v, cand[t].idx);
    free(cand);
    return f;
}

/* ------------------------------------------------------------------ lifetime */
gso_sampler* gso_create(int64_t num_nodes, const int64_t* indptr, const int32_t* indices,
                        int32_t num_hops, const int32_t* fanouts, int32_t cache_width,
                        uint64_t seed, int32_t shared) {
    if (num_nodes <= 0 || num_nodes >= ((int64_t)1 << 31) || !indptr || !fanouts) return NULL;
    if (num_hops < 1 || num_hops > GSO_MAX_HOPS || cache_width < 1 || cache_width > 64) return NULL;
    for (int32_t l = 0; l < num_hops; ++l)
        if (fanouts[l] < 1 || fanouts[l] > cache_width) return NULL;
    gso_sampler* s = (gso_sampler*)calloc(1, sizeof(gso_sampler));
    s->N = num_nodes; s->indptr = indptr; s->indices = indices;
    s->L = num_hops; s->W = cache_width; s->seed = seed; s->shared = shared ? 1 : 0;
    s->theta = -1;
    memcpy(s->fanouts, fanouts, (size_t)num_hops * sizeof(int32_t));
    s->num_caches = s->shared ? 1 : num_hops;
    for (int32_t c = 0; c < s->num_caches; ++c) s->rows[c] = (int32_t**)calloc((size_t)num_nodes, sizeof(int32_t*));
    s->pos = (int32_t*)malloc((size_t)num_nodes * sizeof(int32_t));
    for (int64_t v = 0; v < num_nodes; ++v) s->pos[v] = -1;
    return s;
}

static void free_batch(gso_sampler* s) {
    for (int32_t l = 0; l < GSO_MAX_HOPS; ++l) {
        free(s->blk_indptr[l]); free(s->blk_indices[l]); free(s->blk_picked[l]);
        s->blk_indptr[l] = s->blk_indices[l] = s->blk_picked[l] = NULL;
    }
    free(s->frontier); s->frontier = NULL; s->frontier_cap = 0;
}

void gso_destroy(gso_sampler* s) {
    if (!s) return;
    free_batch(s);
    for (int32_t c = 0; c < s->num_caches; ++c) {
        for (int64_t v = 0; v < s->N; ++v) free(s->rows[c][v]);
        free(s->rows[c]);
    }
    free(s->pos);
    free(s);
}

void gso_set_key_fn(gso_sampler* s, gso_key_fn fn, void* ctx) { s->key_fn = fn; s->key_ctx = ctx; }
void gso_set_theta(gso_sampler* s, int64_t theta) { s->theta = theta < 0 ? -1 : theta; }

static int bad_node(const gso_sampler* s, int32_t layer, int32_t v) {
    return !s || layer < 0 || layer >= s->L || v < 0 || v >= s->N;
}

int gso_cache_row(gso_sampler* s, int32_t layer, int32_t v, int32_t* out) {
    if (bad_node(s, layer, v) || !out) return 1;
    memcpy(out, row_of(s, layer, v), (size_t)s->W * sizeof(int32_t));
    return 0;
}

int gso_cache_set_row(gso_sampler* s, int32_t layer, int32_t v, const int32_t* row) {
    if (bad_node(s, layer, v) || !row) return 1;
    memcpy(row_of(s, layer, v), row, (size_t)s->W * sizeof(int32_t));
    return 0;
}

int gso_refresh_node(gso_sampler* s, int32_t layer, int32_t v, uint32_t step, int32_t r) {
    if (bad_node(s, layer, v) || r < 0 || r > s->W) return 1;
    refresh_row(s, layer, v, step, r);
    return 0;
}

/* The refresh as Algorithms 2 and 3 state it (their periodic branch: RefreshCache / CacheRefresh over
 * all layers): every row of every layer's cache, not only the rows of the batch's frontier.
 * With a dense/sparse split only the dense part has rows. */
int gso_refresh_all(gso_sampler* s, int mode, double gamma, uint32_t step) {
    if (!s || step == 0) return 1;
    if (mode != GSO_MODE_FCR && mode != GSO_MODE_OTF) return 1;
    if (mode == GSO_MODE_OTF && !(gamma >= 0.0 && gamma <= 1.0)) return 1;
    int32_t r = gso_refresh_count(mode, gamma, s->W);
    int32_t caches = s->shared ? 1 : s->L;
    for (int32_t layer = 0; layer < caches; ++layer)
        for (int64_t v = 0; v < s->N; ++v)
            if (degree(s, (int32_t)v) > s->theta) refresh_row(s, layer, (int32_t)v, step, r);
    return 0;
}

int gso_fbl_node(gso_sampler* s, int32_t layer, int32_t v, uint32_t step, int32_t* out, int32_t* count) {
    if (bad_node(s, layer, v) || !out || !count) return 1;
    *count = fbl_row(s, layer, v, step, out);
    return 0;
}

int gso_fetch_node(gso_sampler* s, int32_t layer, int32_t v, uint32_t step, int32_t n_fetch, int32_t* out,
                   int32_t* count) {
    if (bad_node(s, layer, v) || !out || !count || n_fetch < 0) return 1;
    *count = fetch_row(s, layer, v, step, n_fetch, out);
    return 0;
}

int gso_pick_node(gso_sampler* s, int32_t layer, int32_t v, uint32_t step, int32_t* out, int32_t* count) {
    if (bad_node(s, layer, v) || !out || !count) return 1;
    *count = pick_row(s, layer, v, step, out);
    return 0;
}

/* ------------------------------------------------------------------ one batch */
/* SampleBlocks (Algorithms 2 and 3) with the refresh applied to the frontier's own rows:
 * for k = 0..L-1 (layer l = L-1-k): refresh each frontier node's row, pick from it, then
 * relabel: frontier_{k+1} = frontier_k followed by the unseen picked ids in row-major order. */
int gso_sample_batch(gso_sampler* s, const int32_t* seeds, int32_t num_seeds, int mode, double gamma, uint32_t step) {
    if (!s || !seeds || num_seeds < 1 || step == 0) return 1;
    if (mode != GSO_MODE_FCR && mode != GSO_MODE_OTF && mode != GSO_MODE_FBL && mode != GSO_MODE_OTF_FETCH) return 2;
    if ((mode == GSO_MODE_OTF || mode == GSO_MODE_OTF_FETCH) && !(gamma >= 0.0 && gamma <= 1.0)) return 1;
    for (int32_t p = 0; p < num_seeds; ++p)
        if (seeds[p] < 0 || seeds[p] >= s->N) return 3;
    int32_t r = gso_refresh_count(mode, gamma, s->W);

    /* clear the previous batch */
    if (s->frontier)
        for (int32_t p = 0; p < s->n[s->L]; ++p) s->pos[s->frontier[p]] = -1;
    free_batch(s);
    s->stat_refreshed = s->stat_scanned = 0;

    int64_t cap = num_seeds;
    for (int32_t k = 0; k < s->L; ++k) {
        cap += cap * s->fanouts[s->L - 1 - k];
        if (cap > s->N) cap = s->N;
    }
    s->frontier = (int32_t*)malloc((size_t)cap * sizeof(int32_t));
    s->frontier_cap = cap;
    for (int32_t p = 0; p < num_seeds; ++p) {
        if (s->pos[seeds[p]] != -1) { /* duplicate seed: contract violation */
            for (int32_t q = 0; q < p; ++q) s->pos[seeds[q]] = -1;
            free_batch(s);
            return 4;
        }
        s->frontier[p] = seeds[p];
        s->pos[seeds[p]] = p;
    }
    s->n[0] = num_seeds;

    for (int32_t k = 0; k < s->L; ++k) {
        int32_t l = s->L - 1 - k;
        int32_t f = s->fanouts[l];
        int32_t nk = s->n[k];
        int32_t refresh_from = (s->shared && k > 0) ? s->n[k - 1] : 0;
        int32_t* indptr = (int32_t*)malloc(((size_t)nk + 1) * sizeof(int32_t));
        int32_t* picked = (int32_t*)malloc((size_t)nk * (size_t)f * sizeof(int32_t) + 4);
        int32_t* local = (int32_t*)malloc((size_t)nk * (size_t)f * sizeof(int32_t) + 4);
        int32_t m = 0;
        for (int32_t p = 0; p < nk; ++p) {
            int32_t v = s->frontier[p];
            indptr[p] = m;
            /* Dense/sparse split (paper Section "Graph Splitting and Sampling Strategies"): nodes with
             * degree <= theta form the sparse part and are sampled straight from the graph (FBL)
             * in every mode; only the dense part is cached, refreshed and sampled from the cache. */
            if (mode == GSO_MODE_FBL || degree(s, v) <= s->theta) {
                m += fbl_row(s, l, v, step, picked + m);
                continue;
            }
            if (mode == GSO_MODE_OTF_FETCH) {
                m += fetch_row(s, l, v, step, gso_fetch_count(gamma, f), picked + m);
                continue;
            }
            if (p >= refresh_from) refresh_row(s, l, v, step, r);
            m += pick_row(s, l, v, step, picked + m);
        }
        indptr[nk] = m;
        int32_t nn = nk;
        for (int32_t e = 0; e < m; ++e) {
            int32_t u = picked[e];
            if (s->pos[u] == -1) {
                s->pos[u] = nn;
                s->frontier[nn++] = u;
            }
            local[e] = s->pos[u];
        }
        s->n[k + 1] = nn;
        s->m[l] = m;
        s->blk_indptr[l] = indptr;
        s->blk_indices[l] = local;
        s->blk_picked[l] = picked;
    }
    return 0;
}

int32_t gso_num_nodes(const gso_sampler* s, int32_t k) { return (k < 0 || k > s->L) ? -1 : s->n[k]; }
int32_t gso_num_edges(const gso_sampler* s, int32_t layer) { return (layer < 0 || layer >= s->L) ? -1 : s->m[layer]; }
const int32_t* gso_frontier(const gso_sampler* s) { return s->frontier; }
const int32_t* gso_block_indptr(const gso_sampler* s, int32_t layer) { return s->blk_indptr[layer]; }
const int32_t* gso_block_indices(const gso_sampler* s, int32_t layer) { return s->blk_indices[layer]; }
const int32_t* gso_block_picked(const gso_sampler* s, int32_t layer) { return s->blk_picked[layer]; }
int64_t gso_stat_refreshed(const gso_sampler* s) { return s->stat_refreshed; }
int64_t gso_stat_scanned(const gso_sampler* s) { return s->stat_scanned; }

/* ------------------------------------------------------------------ feature gather */
void gso_gather(const void* X, int64_t ld_bytes, int64_t row_bytes, const int32_t* ids, int64_t n,
                void* out, int64_t out_ld_bytes) {
    for (int64_t p = 0; p < n; ++p)
        memcpy((char*)out + p * out_ld_bytes, (const char*)X + (int64_t)ids[p] * ld_bytes, (size_t)row_bytes);
}
