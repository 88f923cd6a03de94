"""TEST INFRASTRUCTURE ONLY: a plain restatement of the paper's prefix-cache bookkeeping, used to check
the library's cp_trie_* calls.  Nothing in the product path may import this file.

What it restates, in the paper's notation:
  * the prefix trie of Section 7.1: one node per cache block, the path from the root is the prefix; every
    node records which workers hold the complete prefix ending there, and per supported CP degree the
    statistics access[z, C] and missed[z, C];
  * ReplicaCount(z, C), MatchedPath(i), ReusedPath(i, w);
  * Eq. 2 (predicted prefill time) and PreferDegree(i): the argmin of the placement cost of Section 5.3
    without its queueing term;
  * Algorithm 1 (per-request statistics update) and Algorithm 2 (periodic scan with decay);
  * the ranking rules stated after Algorithm 2 (inter: missed per copied block, descending; intra:
    access per replica, descending, smaller footprint first on ties; reclaim: access per replica,
    ascending; a bounded number of each).

Dictionaries and lists only; nodes are numbered in creation order (root = 0), children are visited in
creation order, so that lists come out in a defined order.  Pinned by tests/test_oracle_cache_manager.py.
"""
from __future__ import annotations


def remaining_workload(R, P):
    """Eq. 1."""
    return R * P + R * (R + 1) / 2.0


def prefill_time(model, R, P, C):
    """Eq. 2; model = (d, a, b, c, alpha)."""
    d, a, b, c, alpha = model
    return d + a * R + b * P + (c * R + alpha * remaining_workload(R, P)) / C


def prefer_degree(model, L, workers, beta, lam):
    """workers: list of (degree, reused prefix length at that worker).  Cost of Section 5.3 without q_w:
    beta*s + lam*(C_w*s - C_min*E_{C_min}(R_w, P_w)), s = E_{C_w}(R_w, P_w), R_w = L - P_w.
    Returns (index of the first minimum, its degree)."""
    c_min = min(c for c, _ in workers)
    best, best_cost = -1, None
    for i, (c, p) in enumerate(workers):
        s = prefill_time(model, L - p, p, c)
        cost = beta * s + lam * (c * s - c_min * prefill_time(model, L - p, p, c_min))
        if best_cost is None or cost < best_cost:
            best, best_cost = i, cost
    return best, workers[best][0]


class Trie:
    def __init__(self, degrees, block_tokens=64):
        self.degrees = list(degrees)
        self.block = block_tokens
        self.parent = [-1]
        self.depth = [0]
        self.children = [dict()]
        self.holders = [set()]
        self.access = [dict((c, 0.0) for c in self.degrees)]
        self.missed = [dict((c, 0.0) for c in self.degrees)]
        self.worker_degree = {}

    # ---- structure -------------------------------------------------------------------------
    def set_worker(self, worker, degree):
        """Register a worker at a degree; degree 0 removes it and every holder record it had."""
        if degree == 0:
            self.worker_degree.pop(worker, None)
            for h in self.holders:
                h.discard(worker)
        else:
            assert degree in self.degrees
            self.worker_degree[worker] = degree

    def _child(self, z, key, create):
        c = self.children[z].get(key)
        if c is None and create:
            c = len(self.parent)
            self.parent.append(z)
            self.depth.append(self.depth[z] + 1)
            self.children.append(dict())
            self.holders.append(set())
            self.access.append(dict((d, 0.0) for d in self.degrees))
            self.missed.append(dict((d, 0.0) for d in self.degrees))
            self.children[z][key] = c
        return c

    def add_replica(self, blocks, worker):
        """The worker now holds the complete prefix `blocks`: it becomes a holder of every node on the path."""
        assert worker in self.worker_degree
        z = 0
        for key in blocks:
            z = self._child(z, key, True)
            self.holders[z].add(worker)
        return z

    def drop_replica(self, z, worker):
        """Remove the worker's replica of node z; refused (False) if the worker retains a descendant of z."""
        if z <= 0 or worker not in self.holders[z]:
            return False
        if any(worker in self.holders[c] for c in self.children[z].values()):
            return False
        self.holders[z].discard(worker)
        return True

    def replica_count(self, z, C):
        return sum(1 for w in self.holders[z] if self.worker_degree.get(w) == C)

    def prefix_length(self, z):
        return self.depth[z] * self.block

    def matched_path(self, blocks):
        path, z = [], 0
        for key in blocks:
            z = self._child(z, key, False)
            if z is None:
                break
            path.append(z)
        return path

    def reused_path(self, blocks, worker):
        return [z for z in self.matched_path(blocks) if worker in self.holders[z]]

    # ---- Algorithm 1 -----------------------------------------------------------------------
    def update(self, blocks, L, worker, pref_degree, model):
        cw = self.worker_degree[worker]
        for z in self.reused_path(blocks, worker):
            self.access[z][cw] += 1.0
        for z in self.matched_path(blocks):
            if self.replica_count(z, pref_degree) == 0:
                p0 = self.prefix_length(self.parent[z])
                p1 = self.prefix_length(z)
                benefit = prefill_time(model, L - p0, p0, pref_degree) - prefill_time(model, L - p1, p1, pref_degree)
                self.missed[z][pref_degree] += benefit

    # ---- Algorithm 2 and the ranking that follows it ---------------------------------------
    def footprint(self, z, C):
        """Fewest blocks to copy so that some degree-C worker without z holds the path root..z; 0 if there
        is no such worker."""
        path = []
        y = z
        while y > 0:
            path.append(y)
            y = self.parent[y]
        best = 0
        for w, c in sorted(self.worker_degree.items()):
            if c != C or w in self.holders[z]:
                continue
            missing = sum(1 for y in path if w not in self.holders[y])
            if best == 0 or missing < best:
                best = missing
        return best

    def scan(self, theta_inter, theta_intra, theta_reclaim, decay, max_ops):
        inter, intra, reclaim = [], [], []
        for z in range(1, len(self.parent)):
            for C in self.degrees:
                r = self.replica_count(z, C)
                if r == 0:
                    if self.missed[z][C] > theta_inter:
                        fp = self.footprint(z, C)
                        inter.append((z, C, r, fp, self.missed[z][C] / max(fp, 1)))
                else:
                    if self.access[z][C] > r * theta_intra:
                        intra.append((z, C, r, self.footprint(z, C), self.access[z][C] / r))
                    elif self.access[z][C] < r * theta_reclaim:
                        reclaim.append((z, C, r, 0, self.access[z][C] / r))
        for z in range(len(self.parent)):
            for C in self.degrees:
                self.access[z][C] *= decay
                self.missed[z][C] *= decay
        totals = (len(inter), len(intra), len(reclaim))
        inter.sort(key=lambda t: (-t[4], t[0], t[1]))
        intra.sort(key=lambda t: (-t[4], t[3], t[0], t[1]))
        reclaim.sort(key=lambda t: (t[4], t[0], t[1]))
        return inter[:max_ops], intra[:max_ops], reclaim[:max_ops], totals
