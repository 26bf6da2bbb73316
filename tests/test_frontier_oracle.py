"""Pins of the frontier-scheduler oracle against what the paper and plain graph facts fix (no GPU, no product code)."""
import itertools

import numpy as np
import pytest

from oracle import frontier_oracle as FO
from oracle import medverse_oracle as MO


def _random_dag(rng, n, max_parents=3, n_roots=1):
    parents = [[] for _ in range(n)]
    for v in range(n_roots, n):
        k = int(rng.integers(1, min(max_parents, v) + 1))
        parents[v] = sorted(rng.choice(v, size=k, replace=False).tolist())
    return parents


def _longest_path_from_roots(parents):
    """Length of the longest chain of edges ending in each node, by enumerating every path (brute force)."""
    def longest(v):
        return 0 if not parents[v] else 1 + max(longest(p) for p in parents[v])
    return [longest(v) for v in range(len(parents))]


def _run(parents, tokens, ps=16, pages=4096, finished=None):
    s = FO.Scheduler(ps, pages)
    s.add_request(parents, tokens)
    rq = s.requests[0]
    fired_at, trace = {}, []
    for t in rq.running:
        fired_at[t] = rq.k
    while True:
        b = s.step()
        if b is None:
            break
        trace.append(b)
        s.commit(finished(b) if finished else None)
        for t in rq.running:
            fired_at.setdefault(t, rq.k)
    return s, rq, fired_at, trace


def test_worked_example_frontiers_fork_and_join():
    # R -> A, R -> B (diverging edges: two transitions), A, B -> C (converging edges: one transition), R -> D,
    # C, D -> E: the frontiers are {A, B, D}, {C}, {E}  (Eq. 1; Sec. 3.2 on edge aggregation)
    R, A, B, C, D, E = range(6)
    parents = [[], [R], [R], [A, B], [R], [C, D]]
    tokens = [40, 3, 5, 2, 4, 1]
    s, rq, fired_at, trace = _run(parents, tokens)
    assert fired_at == {A: 0, B: 0, D: 0, C: 1, E: 2}
    # barrier: the first frontier takes max(3, 5, 4) steps, then 2, then 1
    assert len(trace) == 5 + 2 + 1
    assert [len(b["row_node"]) for b in trace] == [3, 3, 3, 2, 1, 1, 1, 1]
    assert s.stats["transitions_fired"] == 5 and s.stats["joins"] == 2 and s.stats["forks"] == 3
    assert s.stats["markings_advanced"] == 3
    # a join reads the union of its predecessors' histories: C sees R, A, B; E sees everything before it
    assert rq.view(C) == {R, A, B} and rq.view(E) == {R, A, B, C, D}
    # the rows of the first step and what they may read
    b0 = trace[0]
    assert b0["row_node"] == [A, B, D] and b0["node_new"] == [0, 1, 1, 1] and b0["node_len"] == [40, 0, 0, 0]
    # step 4 (A and D finished earlier, B still running): only B's path is shown
    b4 = trace[4]
    assert b4["row_node"] == [B] and b4["node_len"] == [40, 4]


def test_fork_shares_pages_by_reference_and_join_copies_nothing():
    R, A, B, C = range(4)
    s = FO.Scheduler(16, 64)
    s.add_request([[], [R], [R], [A, B]], [40, 17, 2, 3])
    rq = s.requests[0]
    prefix_pages = list(rq.pages[R])
    assert prefix_pages == [0, 1, 2]  # ceil(40 / 16) pages, lowest ids first
    # Fork: both siblings hold the prefix, which is owned once: 1 + 2 references, and no page was added for it
    assert [s.refs[p] for p in prefix_pages] == [3, 3, 3] and s.stats["pages_in_use"] == 3
    b = s.step()
    assert b["page_idx"] == [0, 1, 2, 3, 4]  # prefix, then the first page of A and of B
    s.commit()
    s.step(); s.commit()  # B is complete after two tokens and lets go of the prefix; A runs on
    assert [s.refs[p] for p in prefix_pages] == [2, 2, 2]
    for _ in range(15):
        s.step(); s.commit()
    # A has 17 tokens: two pages.  The barrier has passed, C (a join) runs and holds R, A, B by reference
    in_use_before = s.stats["pages_in_use"]
    assert rq.k == 1 and set(rq.running) == {C}
    assert in_use_before == 3 + 2 + 1  # firing the join allocated nothing
    assert all(s.refs[p] == 2 for u in (R, A, B) for p in rq.pages[u])
    b = s.step()
    shown_pages = b["page_idx"]
    assert sorted(shown_pages) == sorted(set(shown_pages))  # every page listed once: a union, not a concatenation of copies
    assert shown_pages[:6] == rq.pages[R] + rq.pages[A] + rq.pages[B]
    s.commit(); s.step(); s.commit(); s.step(); s.commit()
    assert rq.done and s.stats["pages_in_use"] == 0 and sorted(s.free) == list(range(64)) and not s.refs


@pytest.mark.parametrize("seed", range(12))
def test_frontier_index_is_longest_path_and_each_step_runs_once(seed):
    rng = np.random.default_rng(seed)
    n = int(rng.integers(2, 11))
    parents = _random_dag(rng, n, n_roots=int(rng.integers(1, 3)) if n > 2 else 1)
    tokens = [int(rng.integers(0, 50)) if not parents[v] else int(rng.integers(1, 9)) for v in range(n)]
    s, rq, fired_at, trace = _run(parents, tokens)
    depth = _longest_path_from_roots(parents)
    transitions = [v for v in range(n) if parents[v]]
    # with the barrier, step v fires under marking M_{depth(v) - 1}
    assert fired_at == {v: depth[v] - 1 for v in transitions}
    assert s.stats["transitions_fired"] == len(transitions)
    # the same layering as the attention oracle's (Eq. 1 read as a recurrence)
    assert [int(x) for x in MO.node_layers(parents)] == depth
    # decode steps: every frontier lasts as long as its longest step
    want_steps = sum(max(tokens[v] for v in transitions if depth[v] == k) for k in sorted({depth[v] for v in transitions}))
    assert len(trace) == want_steps
    # rows of a step = steps still running; every (node, token) is emitted exactly once
    emitted = sorted((v, l) for b in trace for v, l in zip(b["row_node"], [b["node_len"][i] for i, nw in enumerate(b["node_new"]) if nw]))
    assert emitted == sorted((v, j) for v in transitions for j in range(tokens[v]))
    # pages: nothing is freed before the request ends, everything after
    assert s.stats["pages_peak"] == sum(-(-tokens[v] // 16) for v in range(n))
    assert rq.done and s.stats["pages_in_use"] == 0 and not s.refs


def test_linear_chain_is_plain_autoregressive_decoding():
    parents = [[], [0], [1], [2]]
    s, rq, fired_at, trace = _run(parents, [10, 4, 3, 2])
    assert all(len(b["row_node"]) == 1 for b in trace) and len(trace) == 9
    assert s.stats["forks"] == 0 and s.stats["joins"] == 0
    # the single row always reads the whole chain so far
    assert [sum(b["node_len"]) for b in trace] == list(range(10, 19))


def test_emitted_batches_are_valid_planner_input_and_rows_see_their_view():
    rng = np.random.default_rng(5)
    parents = _random_dag(rng, 9)
    tokens = [33] + [int(rng.integers(1, 6)) for _ in range(8)]
    s, rq, fired_at, trace = _run(parents, tokens)
    for b in trace:
        n = b["node_off"][1]
        local_parents = [b["parent_idx"][b["parent_off"][v]:b["parent_off"][v + 1]] for v in range(n)]
        assert all(p < v for v in range(n) for p in local_parents[v])  # topological numbering survives the renumbering
        for v in range(n):
            need = -(-(b["node_len"][v] + b["node_new"][v]) // 16)
            assert b["page_off"][v + 1] - b["page_off"][v] == need
        # a node is shown only if some running step reads it
        layer = MO.node_layers(local_parents)
        vis = MO.visible_sets(local_parents, layer)
        rows = [v for v in range(n) if b["node_new"][v]]
        assert set().union(*[set(vis[v]) for v in rows]) == set(range(n))


def test_early_finish_flag_ends_a_step_and_out_of_pages_is_an_error():
    s = FO.Scheduler(16, 8)
    s.add_request([[], [0], [0]], [16, 100, 100])
    b = s.step()
    assert b["row_node"] == [1, 2]
    s.commit([True, False])  # the engine saw the end of step 1 after one token
    assert s.requests[0].tokens[1] == 1 and set(s.requests[0].running) == {2}
    with pytest.raises(MemoryError):
        for _ in range(200):
            s.step(); s.commit()


def test_two_requests_interleave_and_release_independently():
    s = FO.Scheduler(16, 64)
    s.add_request([[], [0], [0]], [20, 2, 1])
    s.add_request([[], [0]], [5, 4])
    b = s.step()
    assert b["n_req"] == 2 and b["row_req"] == [0, 0, 1] and b["row_node"] == [1, 2, 1]
    s.commit(); s.step(); s.commit()  # request 0 is complete and gone, request 1 runs on
    assert s.requests[0].done and not s.requests[1].done
    b = s.step()
    assert b["n_req"] == 1 and b["row_req"] == [1]
    # request 0's pages (ids 0, 1 and its two step pages) are free again; request 1 still holds its own
    assert s.stats["pages_in_use"] == 2
