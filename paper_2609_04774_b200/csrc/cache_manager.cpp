// Prefix-cache bookkeeping (host only): the global prefix trie with per-degree demand statistics,
// Algorithm 1 (per-request update), Algorithm 2 (periodic scan) with its ranking rules, the
// prefill-time model of Eq. 2 and PreferDegree.  See include/cpcache.h for the contract.
#include <algorithm>
#include <cmath>
#include <cstdint>
#include <limits>
#include <new>
#include <unordered_map>
#include <vector>

#include "cpcache.h"
#include "internal.h"

using cpattn::set_error;

namespace {

struct EdgeKey {
    int32_t parent;
    uint64_t block;
    bool operator==(const EdgeKey& o) const { return parent == o.parent && block == o.block; }
};
struct EdgeHash {
    size_t operator()(const EdgeKey& k) const {
        uint64_t x = k.block ^ (0x9E3779B97F4A7C15ull * (uint64_t)(uint32_t)(k.parent + 1));
        x ^= x >> 31; x *= 0xBF58476D1CE4E5B9ull; x ^= x >> 29;
        return (size_t)x;
    }
};

struct Node {
    int32_t parent;
    int32_t depth;
    int32_t first_child;
    int32_t last_child;
    int32_t next_sibling;
    std::vector<int32_t> holders;   // sorted worker ids
};

inline double workload(int64_t R, int64_t P) {   // Eq. 1
    return (double)R * (double)P + (double)R * ((double)R + 1.0) / 2.0;
}

inline double predict(const cp_prefill_model& m, int64_t R, int64_t P, int32_t C) {   // Eq. 2
    return m.d + m.a * (double)R + m.b * (double)P + (m.c * (double)R + m.alpha * workload(R, P)) / (double)C;
}

}  // namespace

struct cp_trie {
    std::vector<int32_t> degrees;
    int32_t block_tokens;
    std::vector<Node> nodes;
    std::unordered_map<EdgeKey, int32_t, EdgeHash> edges;
    std::vector<double> access, missed;                 // [node][degree index]
    std::unordered_map<int32_t, int32_t> worker_degree; // worker -> degree

    int degree_index(int32_t C) const {
        for (size_t i = 0; i < degrees.size(); ++i)
            if (degrees[i] == C) return (int)i;
        return -1;
    }
    int32_t child(int32_t z, uint64_t key) const {
        auto it = edges.find(EdgeKey{z, key});
        return it == edges.end() ? -1 : it->second;
    }
    int32_t make_child(int32_t z, uint64_t key) {
        const int32_t c = (int32_t)nodes.size();
        nodes.push_back(Node{z, nodes[z].depth + 1, -1, -1, -1, {}});
        // children are kept in creation order: append at the tail of the sibling list
        if (nodes[z].first_child < 0) nodes[z].first_child = c;
        else nodes[nodes[z].last_child].next_sibling = c;
        nodes[z].last_child = c;
        edges.emplace(EdgeKey{z, key}, c);
        access.resize(nodes.size() * degrees.size(), 0.0);
        missed.resize(nodes.size() * degrees.size(), 0.0);
        return c;
    }
    bool holds(int32_t z, int32_t worker) const {
        return std::binary_search(nodes[z].holders.begin(), nodes[z].holders.end(), worker);
    }
    int32_t replica_count(int32_t z, int32_t C) const {
        int32_t n = 0;
        for (int32_t w : nodes[z].holders) {
            auto it = worker_degree.find(w);
            if (it != worker_degree.end() && it->second == C) ++n;
        }
        return n;
    }
    // Fewest missing blocks on the path root..z over the degree-C workers that lack z; 0 if none lacks it.
    int32_t footprint(int32_t z, int32_t C) const {
        int32_t best = 0;
        for (const auto& wd : worker_degree) {
            if (wd.second != C || holds(z, wd.first)) continue;
            int32_t missing = 0;
            for (int32_t y = z; y > 0; y = nodes[y].parent)
                if (!holds(y, wd.first)) ++missing;
            if (best == 0 || missing < best) best = missing;
        }
        return best;
    }
};

extern "C" double cp_prefill_time(const cp_prefill_model* model, int64_t R, int64_t P, int32_t C) {
    if (!model || C < 1) return std::numeric_limits<double>::quiet_NaN();
    return predict(*model, R, P, C);
}

extern "C" int cp_prefer_degree(const cp_prefill_model* model, int64_t L, int32_t n, const int32_t* degree,
                                const int64_t* reused_len, double beta, double lambda, int32_t* worker_out,
                                int32_t* degree_out) {
    if (!model || !degree || !reused_len || !worker_out || !degree_out || n < 1 || L < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_prefer_degree: null pointer, n < 1 or L < 1");
    int32_t c_min = std::numeric_limits<int32_t>::max();
    for (int32_t i = 0; i < n; ++i) {
        if (degree[i] < 1 || reused_len[i] < 0 || reused_len[i] > L)
            return set_error(CP_ERR_INVALID_ARG, "cp_prefer_degree: worker %d has degree %d, reused_len %lld (L = %lld)", i,
                             degree[i], (long long)reused_len[i], (long long)L);
        c_min = std::min(c_min, degree[i]);
    }
    int32_t best = -1;
    double best_cost = 0.0;
    for (int32_t i = 0; i < n; ++i) {
        const int64_t P = reused_len[i], R = L - P;
        const double s = predict(*model, R, P, degree[i]);
        const double cost = beta * s + lambda * ((double)degree[i] * s - (double)c_min * predict(*model, R, P, c_min));
        if (best < 0 || cost < best_cost) {
            best = i;
            best_cost = cost;
        }
    }
    *worker_out = best;
    *degree_out = degree[best];
    return CP_OK;
}

extern "C" int cp_trie_create(cp_trie** out, const int32_t* degrees, int32_t n_degrees, int32_t block_tokens) {
    if (!out || !degrees || n_degrees < 1 || block_tokens < 1)
        return set_error(CP_ERR_INVALID_ARG, "cp_trie_create: null pointer, no degrees or block_tokens < 1");
    for (int32_t i = 0; i < n_degrees; ++i) {
        if (degrees[i] < 1) return set_error(CP_ERR_INVALID_ARG, "cp_trie_create: degree %d", degrees[i]);
        for (int32_t j = 0; j < i; ++j)
            if (degrees[j] == degrees[i]) return set_error(CP_ERR_INVALID_ARG, "cp_trie_create: degree %d listed twice", degrees[i]);
    }
    cp_trie* t = new (std::nothrow) cp_trie();
    if (!t) return set_error(CP_ERR_INVALID_ARG, "cp_trie_create: out of host memory");
    t->degrees.assign(degrees, degrees + n_degrees);
    t->block_tokens = block_tokens;
    t->nodes.push_back(Node{-1, 0, -1, -1, -1, {}});
    t->access.assign(t->degrees.size(), 0.0);
    t->missed.assign(t->degrees.size(), 0.0);
    *out = t;
    return CP_OK;
}

extern "C" int cp_trie_destroy(cp_trie* t) {
    delete t;
    return CP_OK;
}

extern "C" int cp_trie_set_worker(cp_trie* t, int32_t worker, int32_t degree) {
    if (!t || worker < 0) return set_error(CP_ERR_INVALID_ARG, "cp_trie_set_worker: null trie or negative worker id");
    if (degree == 0) {
        t->worker_degree.erase(worker);
        for (Node& n : t->nodes) {
            auto it = std::lower_bound(n.holders.begin(), n.holders.end(), worker);
            if (it != n.holders.end() && *it == worker) n.holders.erase(it);
        }
        return CP_OK;
    }
    if (t->degree_index(degree) < 0) return set_error(CP_ERR_INVALID_ARG, "cp_trie_set_worker: degree %d is not supported", degree);
    t->worker_degree[worker] = degree;
    return CP_OK;
}

extern "C" int cp_trie_add_replica(cp_trie* t, const uint64_t* blocks, int32_t n, int32_t worker, int32_t* node_out) {
    if (!t || !blocks || n < 1) return set_error(CP_ERR_INVALID_ARG, "cp_trie_add_replica: null pointer or n < 1");
    if (!t->worker_degree.count(worker)) return set_error(CP_ERR_INVALID_ARG, "cp_trie_add_replica: unknown worker %d", worker);
    int32_t z = 0;
    for (int32_t i = 0; i < n; ++i) {
        int32_t c = t->child(z, blocks[i]);
        if (c < 0) c = t->make_child(z, blocks[i]);
        z = c;
        auto& h = t->nodes[z].holders;
        auto it = std::lower_bound(h.begin(), h.end(), worker);
        if (it == h.end() || *it != worker) h.insert(it, worker);
    }
    if (node_out) *node_out = z;
    return CP_OK;
}

extern "C" int cp_trie_drop_replica(cp_trie* t, int32_t node, int32_t worker) {
    if (!t || node < 1 || node >= (int32_t)t->nodes.size())
        return set_error(CP_ERR_INVALID_ARG, "cp_trie_drop_replica: node %d does not exist", node);
    if (!t->holds(node, worker)) return set_error(CP_ERR_BOUNDS, "cp_trie_drop_replica: worker %d does not hold node %d", worker, node);
    for (int32_t c = t->nodes[node].first_child; c >= 0; c = t->nodes[c].next_sibling)
        if (t->holds(c, worker))
            return set_error(CP_ERR_BOUNDS, "cp_trie_drop_replica: worker %d still retains child %d of node %d", worker, c, node);
    auto& h = t->nodes[node].holders;
    h.erase(std::lower_bound(h.begin(), h.end(), worker));
    return CP_OK;
}

extern "C" int cp_trie_match(const cp_trie* t, const uint64_t* blocks, int32_t n, int32_t* nodes, int32_t* n_matched) {
    if (!t || (!blocks && n > 0) || n < 0 || !n_matched) return set_error(CP_ERR_INVALID_ARG, "cp_trie_match: null pointer or n < 0");
    int32_t z = 0, m = 0;
    for (; m < n; ++m) {
        const int32_t c = t->child(z, blocks[m]);
        if (c < 0) break;
        z = c;
        if (nodes) nodes[m] = z;
    }
    *n_matched = m;
    return CP_OK;
}

extern "C" int cp_trie_reused(const cp_trie* t, const uint64_t* blocks, int32_t n, int32_t worker, int32_t* n_reused) {
    if (!t || (!blocks && n > 0) || n < 0 || !n_reused) return set_error(CP_ERR_INVALID_ARG, "cp_trie_reused: null pointer or n < 0");
    int32_t z = 0, m = 0;
    for (; m < n; ++m) {
        const int32_t c = t->child(z, blocks[m]);
        if (c < 0 || !t->holds(c, worker)) break;
        z = c;
    }
    *n_reused = m;
    return CP_OK;
}

extern "C" int cp_trie_reused_all(const cp_trie* t, const uint64_t* blocks, int32_t n, const int32_t* workers,
                                  int32_t n_workers, int32_t* n_reused) {
    if (!t || (!blocks && n > 0) || n < 0 || !workers || !n_reused || n_workers < 0)
        return set_error(CP_ERR_INVALID_ARG, "cp_trie_reused_all: null pointer or negative count");
    for (int32_t i = 0; i < n_workers; ++i) n_reused[i] = 0;
    // holders hold complete prefixes, so a worker's reused path is a leading part of the matched path
    int32_t z = 0;
    for (int32_t m = 0; m < n; ++m) {
        const int32_t c = t->child(z, blocks[m]);
        if (c < 0) break;
        z = c;
        bool any = false;
        for (int32_t i = 0; i < n_workers; ++i)
            if (n_reused[i] == m && t->holds(z, workers[i])) {
                n_reused[i] = m + 1;
                any = true;
            }
        if (!any) break;
    }
    return CP_OK;
}

extern "C" int cp_trie_replica_count(const cp_trie* t, int32_t node, int32_t degree, int32_t* count) {
    if (!t || !count || node < 0 || node >= (int32_t)t->nodes.size())
        return set_error(CP_ERR_INVALID_ARG, "cp_trie_replica_count: node %d does not exist", node);
    *count = t->replica_count(node, degree);
    return CP_OK;
}

extern "C" int cp_trie_stats(const cp_trie* t, int32_t node, int32_t degree, double* access, double* missed) {
    if (!t || node < 0 || node >= (int32_t)t->nodes.size())
        return set_error(CP_ERR_INVALID_ARG, "cp_trie_stats: node %d does not exist", node);
    const int di = t->degree_index(degree);
    if (di < 0) return set_error(CP_ERR_INVALID_ARG, "cp_trie_stats: degree %d is not supported", degree);
    if (access) *access = t->access[(size_t)node * t->degrees.size() + di];
    if (missed) *missed = t->missed[(size_t)node * t->degrees.size() + di];
    return CP_OK;
}

extern "C" int cp_trie_size(const cp_trie* t, int32_t* n_nodes) {
    if (!t || !n_nodes) return set_error(CP_ERR_INVALID_ARG, "cp_trie_size: null pointer");
    *n_nodes = (int32_t)t->nodes.size();
    return CP_OK;
}

extern "C" int cp_trie_update(cp_trie* t, const uint64_t* blocks, int32_t n, int64_t L, int32_t worker,
                              int32_t pref_degree, const cp_prefill_model* model) {
    if (!t || (!blocks && n > 0) || n < 0 || !model) return set_error(CP_ERR_INVALID_ARG, "cp_trie_update: null pointer or n < 0");
    auto wd = t->worker_degree.find(worker);
    if (wd == t->worker_degree.end()) return set_error(CP_ERR_INVALID_ARG, "cp_trie_update: unknown worker %d", worker);
    const int di_w = t->degree_index(wd->second), di_p = t->degree_index(pref_degree);
    if (di_p < 0) return set_error(CP_ERR_INVALID_ARG, "cp_trie_update: preferred degree %d is not supported", pref_degree);
    const size_t nd = t->degrees.size();
    // matched path first: nothing is modified if the request is inconsistent
    std::vector<int32_t> path;
    int32_t z = 0;
    for (int32_t i = 0; i < n; ++i) {
        const int32_t c = t->child(z, blocks[i]);
        if (c < 0) break;
        z = c;
        path.push_back(z);
    }
    if ((int64_t)path.size() * t->block_tokens > L)
        return set_error(CP_ERR_INVALID_ARG, "cp_trie_update: L = %lld is shorter than the matched prefix of %zu blocks",
                         (long long)L, path.size());
    for (int32_t y : path) {           // reused path: the leading nodes the selected worker holds
        if (!t->holds(y, worker)) break;
        t->access[(size_t)y * nd + di_w] += 1.0;
    }
    for (int32_t y : path) {
        if (t->replica_count(y, pref_degree) != 0) continue;
        const int64_t p1 = (int64_t)t->nodes[y].depth * t->block_tokens, p0 = p1 - t->block_tokens;
        const double benefit = predict(*model, L - p0, p0, pref_degree) - predict(*model, L - p1, p1, pref_degree);
        t->missed[(size_t)y * nd + di_p] += benefit;
    }
    return CP_OK;
}

extern "C" int cp_trie_scan(cp_trie* t, double theta_inter, double theta_intra, double theta_reclaim, double decay,
                            int32_t max_ops, cp_trie_candidate* inter, cp_trie_candidate* intra,
                            cp_trie_candidate* reclaim, int32_t* written, int32_t* totals) {
    if (!t || !written || max_ops < 0 || !(decay > 0.0 && decay <= 1.0) || (max_ops > 0 && (!inter || !intra || !reclaim)))
        return set_error(CP_ERR_INVALID_ARG, "cp_trie_scan: null pointer, max_ops < 0 or decay outside (0, 1]");
    const size_t nd = t->degrees.size();
    std::vector<cp_trie_candidate> li, la, lr;
    for (int32_t z = 1; z < (int32_t)t->nodes.size(); ++z) {
        for (size_t di = 0; di < nd; ++di) {
            const int32_t C = t->degrees[di];
            const int32_t r = t->replica_count(z, C);
            const double acc = t->access[(size_t)z * nd + di], mis = t->missed[(size_t)z * nd + di];
            if (r == 0) {
                if (mis > theta_inter) {
                    const int32_t fp = t->footprint(z, C);
                    li.push_back({z, C, r, fp, mis / (double)std::max(fp, 1)});
                }
            } else if (acc > r * theta_intra) {
                la.push_back({z, C, r, t->footprint(z, C), acc / r});
            } else if (acc < r * theta_reclaim) {
                lr.push_back({z, C, r, 0, acc / r});
            }
        }
    }
    for (double& x : t->access) x *= decay;
    for (double& x : t->missed) x *= decay;
    auto by_node = [](const cp_trie_candidate& a, const cp_trie_candidate& b) {
        return a.node != b.node ? a.node < b.node : a.degree < b.degree;
    };
    std::sort(li.begin(), li.end(), [&](const cp_trie_candidate& a, const cp_trie_candidate& b) {
        return a.score != b.score ? a.score > b.score : by_node(a, b);
    });
    std::sort(la.begin(), la.end(), [&](const cp_trie_candidate& a, const cp_trie_candidate& b) {
        if (a.score != b.score) return a.score > b.score;
        return a.footprint != b.footprint ? a.footprint < b.footprint : by_node(a, b);
    });
    std::sort(lr.begin(), lr.end(), [&](const cp_trie_candidate& a, const cp_trie_candidate& b) {
        return a.score != b.score ? a.score < b.score : by_node(a, b);
    });
    const std::vector<cp_trie_candidate>* lists[3] = {&li, &la, &lr};
    cp_trie_candidate* outs[3] = {inter, intra, reclaim};
    for (int k = 0; k < 3; ++k) {
        const int32_t n = (int32_t)std::min<size_t>(lists[k]->size(), (size_t)max_ops);
        for (int32_t i = 0; i < n; ++i) outs[k][i] = (*lists[k])[i];
        written[k] = n;
        if (totals) totals[k] = (int32_t)lists[k]->size();
    }
    return CP_OK;
}
