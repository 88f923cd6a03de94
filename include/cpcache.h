/* cpcache.h -- prefix-cache bookkeeping of the adaptive-CP serving system: the global prefix trie with
 * its per-degree demand statistics, the per-request update (Algorithm 1), the periodic scan
 * (Algorithm 2) with the ranking rules that follow it, the prefill-time model (Eq. 2) and
 * PreferDegree (Section 7.1).  Host-only integer and double arithmetic; part of libcpattn.so.
 *
 * Conventions as in cpattn.h: every call returns CP_OK (0) or a negative CP_ERR_* code and leaves a
 * message for cp_last_error(); nothing throws across the boundary; all arrays are caller-owned host
 * memory.  A cp_trie is not thread-safe: one manager thread owns it.
 *
 * Nodes are numbered in creation order; node 0 is the root (the empty prefix, not a cache block).
 * Node z at depth k stands for the k-th cache block of a prefix; PrefixLength(z) = k * block_tokens.
 * A block is named by a caller-chosen 64-bit key (for example a hash of its tokens); the path of keys
 * from the root identifies the prefix.
 */
#ifndef CPCACHE_H_
#define CPCACHE_H_

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

/* Eq. 2:  E_C(R, P) = d + a R + b P + (c R + alpha W(R, P)) / C,  W(R, P) = R P + R (R + 1) / 2 (Eq. 1). */
typedef struct { double d, a, b, c, alpha; } cp_prefill_model;

/* Predicted prefill time of R uncached tokens behind P cached ones at CP degree C (Eq. 2).
 * Returns NaN when model is NULL or C < 1. */
double cp_prefill_time(const cp_prefill_model* model, int64_t R, int64_t P, int32_t C);

/* PreferDegree (Section 7.1): the worker minimising the placement cost of Section 5.3 without its
 * queueing term,  beta * s_w + lambda * (C_w * s_w - C_min * E_{C_min}(R_w, P_w)),  where
 * P_w = reused_len[w] is the prefix the worker can reuse, R_w = L - P_w, s_w = E_{C_w}(R_w, P_w) and
 * C_min is the smallest degree among the n workers.  The first minimum wins a tie.
 *   degree, reused_len  host [n];  worker_out / degree_out  receive the index and its degree.
 * Errors: INVALID_ARG (n < 1, a degree < 1, reused_len outside [0, L], NULL pointers). */
int cp_prefer_degree(const cp_prefill_model* model, int64_t L, int32_t n, const int32_t* degree,
                     const int64_t* reused_len, double beta, double lambda, int32_t* worker_out, int32_t* degree_out);

typedef struct cp_trie cp_trie;

/* Creates an empty trie for the supported CP degrees (distinct, >= 1) and a cache block of block_tokens
 * tokens.  Destroy with cp_trie_destroy.  Errors: INVALID_ARG. */
int cp_trie_create(cp_trie** out, const int32_t* degrees, int32_t n_degrees, int32_t block_tokens);
int cp_trie_destroy(cp_trie* t);

/* Registers worker `worker` (any non-negative id) at a supported degree, or moves it to another degree
 * (worker reconfiguration: its holder records are kept and now count for the new degree).  degree 0
 * removes the worker and all its holder records.  Errors: INVALID_ARG (unsupported degree). */
int cp_trie_set_worker(cp_trie* t, int32_t worker, int32_t degree);

/* The worker now holds the complete prefix blocks[0..n): it becomes a holder of every node on the path;
 * missing nodes are created.  node_out (may be NULL) receives the last node.  Errors: INVALID_ARG
 * (unknown worker, n < 1). */
int cp_trie_add_replica(cp_trie* t, const uint64_t* blocks, int32_t n, int32_t worker, int32_t* node_out);

/* Removes the worker's replica of node z.  Refused with CP_ERR_BOUNDS when the worker is not a holder
 * of z or still retains a child of z (a removal must not invalidate retained descendant prefixes). */
int cp_trie_drop_replica(cp_trie* t, int32_t node, int32_t worker);

/* MatchedPath: the nodes of the longest known prefix of blocks[0..n), wherever they are replicated.
 * nodes: host [n] (may be NULL); n_matched receives the count. */
int cp_trie_match(const cp_trie* t, const uint64_t* blocks, int32_t n, int32_t* nodes, int32_t* n_matched);

/* ReusedPath length: how many leading nodes of the matched path the worker holds. */
int cp_trie_reused(const cp_trie* t, const uint64_t* blocks, int32_t n, int32_t worker, int32_t* n_reused);

/* The same for n_workers workers in one call (what a router asks per request): n_reused host [n_workers]. */
int cp_trie_reused_all(const cp_trie* t, const uint64_t* blocks, int32_t n, const int32_t* workers, int32_t n_workers,
                       int32_t* n_reused);

/* ReplicaCount(z, C): holders of node z whose worker is registered at degree C. */
int cp_trie_replica_count(const cp_trie* t, int32_t node, int32_t degree, int32_t* count);

/* access[z, C] and missed[z, C] (either pointer may be NULL); cp_trie_size: number of nodes, root included. */
int cp_trie_stats(const cp_trie* t, int32_t node, int32_t degree, double* access, double* missed);
int cp_trie_size(const cp_trie* t, int32_t* n_nodes);

/* Algorithm 1, for a request of L tokens with block keys blocks[0..n) that was assigned to `worker` and
 * prefers degree pref_degree: access[z, C_worker] += 1 on the reused path; for every node z of the matched
 * path without a replica at pref_degree,
 *   missed[z, pref_degree] += E(L - P0, P0) - E(L - P1, P1) at degree pref_degree,
 * P0 = PrefixLength(Parent(z)), P1 = PrefixLength(z).  Errors: INVALID_ARG (unknown worker, unsupported
 * degree, L shorter than the matched prefix). */
int cp_trie_update(cp_trie* t, const uint64_t* blocks, int32_t n, int64_t L, int32_t worker, int32_t pref_degree,
                   const cp_prefill_model* model);

/* One candidate of a scan.  footprint: fewest blocks to copy so that some degree-`degree` worker that
 * lacks the node holds its whole path (0: no such worker; reclaim candidates: 0).  score: missed per
 * copied block (inter), access per replica (intra, reclaim). */
typedef struct { int32_t node, degree, replicas, footprint; double score; } cp_trie_candidate;

/* Algorithm 2 over every node and supported degree, r = ReplicaCount(z, C):
 *   r == 0 and missed > theta_inter          -> inter-degree replication candidate
 *   r  > 0 and access > r * theta_intra      -> intra-degree replication candidate
 *   r  > 0 and access < r * theta_reclaim    -> reclamation candidate
 * then access and missed of every node are multiplied by decay (0 < decay <= 1).  The lists are ranked
 * (inter: score descending; intra: score descending, smaller footprint first on ties; reclaim: score
 * ascending; remaining ties by node, then degree) and the first max_ops of each are written.
 *   inter / intra / reclaim  host [max_ops] each;  written[3] receives how many were written,
 *   totals[3] (may be NULL) how many candidates each list had before the cut.
 * Errors: INVALID_ARG (decay outside (0, 1], max_ops < 0, NULL arrays with max_ops > 0). */
int cp_trie_scan(cp_trie* t, double theta_inter, double theta_intra, double theta_reclaim, double decay,
                 int32_t max_ops, cp_trie_candidate* inter, cp_trie_candidate* intra, cp_trie_candidate* reclaim,
                 int32_t* written, int32_t* totals);

#ifdef __cplusplus
}
#endif
#endif /* CPCACHE_H_ */
