"""CPU oracle for the frontier scheduler: Petri-net marking, enabled-transition frontier, Fork / Join as
page-table operations.

TEST INFRASTRUCTURE ONLY.  Only the test-suite may import this file; it imports nothing from the product.

The net of one request (Sec. 3.2, "Formal Definition"), in the transition-level form the attention planner takes:
node v of the reasoning DAG owns the place p_v that holds its token once the step is written, and, unless v is a
root, the transition t_v with pre-set {p_u : u parent of v} and post-set {p_v}.  Roots (in-degree zero) are the
places marked by M_0: their text, the context produced before graph execution starts, is already in the KV cache.
Markings only grow: a token stays in its place after the steps that read it have fired (diverging edges are
distinct transitions that all read the same place; Sec. 3.2), and "output place empty" is what makes every step run
exactly once.

What follows the paper and where:
  * enabled-transition frontier F_k: every input place marked, every output place empty      -- Eq. 1
  * all transitions of F_k decode concurrently, one token per decode step each; the marking advances to M_{k+1}
    only when all of them are complete, then the frontier is recomputed                      -- Sec. 3.3, execution loop
  * a token is tau = (h, k): here k, the KV-cache references of a path, is the list of pages of every node the
    step may read; Fork hands the same pages to every sibling (a reference count goes up, nothing is copied); Join
    is the union of the predecessors' lists                                                    -- Sec. 3.2, Sec. 4.3
Readings taken where the paper is silent: a finished step of a frontier that is still running keeps its pages but is
not marked until the barrier; pages are handed out lowest free id first (any policy would do, this one makes the
output unique); a page's reference count is one for the node that owns it plus one for every running step that reads
it; everything a request holds is released when nothing of it is running or enabled.

Everything is written as the definition: Python sets for markings and frontiers, recomputed from scratch, lists for
page tables.
"""
from __future__ import annotations

import heapq


class Request:
    def __init__(self, parents, tokens):
        self.parents = [list(p) for p in parents]
        self.tokens = list(tokens)  # roots: tokens already in the cache; others: tokens the step will emit
        n = len(parents)
        self.places = set(range(n))
        self.transitions = {v for v in range(n) if self.parents[v]}
        self.marked = {v for v in range(n) if not self.parents[v]}  # M_0
        self.running = {}  # transition -> tokens written so far
        self.active = set()  # the frontier being executed (running or waiting at the barrier)
        self.pages = [[] for _ in range(n)]
        self.k = 0  # index of the marking
        self.done = False

    def pre_set(self, t):
        return set(self.parents[t])

    def post_set(self, t):
        return {t}

    def frontier(self):
        """Eq. 1, literally."""
        return {t for t in self.transitions
                if all(p in self.marked for p in self.pre_set(t)) and all(q not in self.marked for q in self.post_set(t))}

    def view(self, t):
        """Nodes a step reads besides itself: the union of its predecessors' histories (Join), which for a single
        predecessor is that predecessor's history (Fork: the same for every sibling)."""
        out = set()
        for p in self.parents[t]:
            out |= {p} | self.view(p)
        return out


class Scheduler:
    def __init__(self, page_size, num_pages):
        self.ps = page_size
        self.free = list(range(num_pages))
        heapq.heapify(self.free)
        self.refs = {}
        self.requests = []
        self.stats = dict(transitions_fired=0, forks=0, joins=0, markings_advanced=0, decode_steps=0, rows_emitted=0,
                          pages_in_use=0, pages_peak=0)

    # ---- pages
    def _alloc(self):
        if not self.free:
            raise MemoryError("out of pages")
        p = heapq.heappop(self.free)
        self.refs[p] = 1  # the owning node
        self.stats["pages_in_use"] += 1
        self.stats["pages_peak"] = max(self.stats["pages_peak"], self.stats["pages_in_use"])
        return p

    def _unref(self, p):
        self.refs[p] -= 1
        assert self.refs[p] >= 0
        if self.refs[p] == 0:
            del self.refs[p]
            heapq.heappush(self.free, p)
            self.stats["pages_in_use"] -= 1

    # ---- requests
    def add_request(self, parents, tokens):
        rq = Request(parents, tokens)
        for v in sorted(rq.marked):
            for _ in range(-(-rq.tokens[v] // self.ps)):
                rq.pages[v].append(self._alloc())
        self.requests.append(rq)
        self._fire(rq)
        return len(self.requests) - 1

    def _fire(self, rq):
        """Activate the frontier of the current marking; release the request if there is none."""
        f = rq.frontier()
        if not f:
            rq.done = True
            for v in sorted(rq.places):
                for p in rq.pages[v]:
                    self._unref(p)
                rq.pages[v] = []
            return
        rq.active = set(f)
        for t in sorted(f):
            rq.running[t] = 0
            self.stats["transitions_fired"] += 1
            if len(rq.parents[t]) >= 2:
                self.stats["joins"] += 1
            if any(sum(1 for s in f if p in rq.parents[s]) >= 2 for p in rq.parents[t]):
                self.stats["forks"] += 1
            for u in rq.view(t):  # the step's references to what it reads: counted, never copied
                for p in rq.pages[u]:
                    self.refs[p] += 1

    # ---- one decode step
    def step(self):
        """The batch of this decode step, as plain lists, or None when nothing is running."""
        node_off, node_len, node_new, parent_off, parent_idx, page_off, page_idx = [0], [], [], [0], [], [0], []
        row_req, row_node = [], []
        n_req = 0
        for r, rq in enumerate(self.requests):
            if rq.done or not rq.running:
                continue
            for t in sorted(rq.running):
                if rq.running[t] % self.ps == 0:  # the token about to be written opens a page
                    rq.pages[t].append(self._alloc())
            shown = set()
            for t in rq.running:
                shown |= {t} | rq.view(t)
            order = sorted(shown)
            local = {v: i for i, v in enumerate(order)}
            for v in order:
                if v in rq.running:
                    node_len.append(rq.running[v]); node_new.append(1)
                    row_req.append(r); row_node.append(v)
                else:
                    node_len.append(rq.tokens[v]); node_new.append(0)
                parent_idx.extend(local[p] for p in rq.parents[v])
                parent_off.append(len(parent_idx))
                page_idx.extend(rq.pages[v])
                page_off.append(len(page_idx))
            node_off.append(len(node_len))
            n_req += 1
        if n_req == 0:
            return None
        self.stats["decode_steps"] += 1
        self.stats["rows_emitted"] += len(row_req)
        return dict(n_req=n_req, node_off=node_off, node_len=node_len, node_new=node_new, parent_off=parent_off,
                    parent_idx=parent_idx, page_off=page_off, page_idx=page_idx, row_req=row_req, row_node=row_node)

    def commit(self, finished=None):
        """Every running step has written one token; `finished[row]` ends a step before its stated length."""
        row = 0
        for rq in self.requests:
            if rq.done or not rq.running:
                continue
            for t in sorted(rq.running):
                rq.running[t] += 1
                if rq.running[t] >= rq.tokens[t] or (finished is not None and finished[row]):
                    rq.tokens[t] = rq.running[t]
                    del rq.running[t]
                    for u in rq.view(t):
                        for p in rq.pages[u]:
                            self._unref(p)
                row += 1
            if not rq.running:  # the barrier: M_{k+1} marks every output place of F_k
                rq.marked |= rq.active
                rq.active = set()
                rq.k += 1
                self.stats["markings_advanced"] += 1
                self._fire(rq)
