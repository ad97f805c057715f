"""Oracle pins: exhaustive schedule searches for tiny problems.

Test infrastructure only.  Nothing here reads the DP tables of ``oracle.policy`` (and this
module does not import it): each search explores the machine of the paper's cost model
directly -- a sequence of ``t`` steps, a memory that holds a bounded number of states, one
working RNN core, forward operations costing 1 and everything else costing 0 (Section 3.1,
definition of ``C(t, m)``) -- and returns the cheapest way to backpropagate all ``t`` steps
in the order t, t-1, ..., 1.

* ``hsm_unrestricted`` / ``ism_unrestricted``: shortest path over *all* machine states; no
  stack discipline, no divide-and-conquer structure is assumed.
* ``msm_protocol``: exhaustive enumeration of every divide-and-conquer tree the protocol of
  Section 3.3 allows, each one *simulated* with a unit counter.  (For the mixed scheme the
  DP is optimal among stack-disciplined schedules only, so that is the space searched.)
"""
from __future__ import annotations

from collections import deque

INFEASIBLE = None


def _zero_one_bfs(start, is_goal, moves):
    """Shortest path with edge costs in {0, 1}."""
    dist = {start: 0}
    dq = deque([start])
    while dq:
        u = dq.popleft()
        du = dist[u]
        if is_goal(u):
            return du
        for v, w in moves(u):
            nd = du + w
            if v not in dist or nd < dist[v]:
                dist[v] = nd
                if w == 0:
                    dq.appendleft(v)
                else:
                    dq.append(v)
    return INFEASIBLE


def hsm_unrestricted(t: int, m: int):
    """Fewest forward operations when memory holds at most ``m`` hidden states.

    State (b, S, p): steps 1..b still await their backward operation; S is the set of stored
    hidden-state positions (position 0, the initial state, is always there and counts as one
    of the m); p is the step whose internal state the working core holds (0 = none).
    The core can run forward from any stored hidden state or from its own output; a backward
    operation over step b needs the core to hold step b and consumes it.
    """
    if m < 1:
        return INFEASIBLE
    start = (t, frozenset([0]), 0)

    def moves(u):
        b, S, p = u
        if b == 0:
            return
        # forward from a stored hidden state q: the core then holds step q + 1
        for q in S:
            if q + 1 <= b:
                yield (b, S, q + 1), 1
        # forward from the core's own output hidden state
        if p and p + 1 <= b:
            yield (b, S, p + 1), 1
        # memorise the core's output hidden state
        if p and p not in S and len(S) < m:
            yield (b, S | {p}, p), 0
        # forget a stored state (never the initial one)
        for q in S:
            if q != 0:
                yield (b, S - {q}, p), 0
        # backward over step b
        if p == b:
            yield (b - 1, frozenset(q for q in S if q < b), 0), 0

    return _zero_one_bfs(start, lambda u: u[0] == 0, moves)


def ism_unrestricted(t: int, m: int):
    """Fewest forward operations when memory holds at most ``m`` internal states.

    State (b, S, p): S = positions whose internal states are stored; p = position of the
    core being computed (0 = none), which occupies one of the m places as well.  The initial
    hidden state is free.  An internal state contains its output hidden state, so a forward
    operation may start from any stored position, from position 0, or from the core itself.
    A backward operation over step b needs b in S or p = b, and releases that state.
    """
    if m < 1:
        return INFEASIBLE
    start = (t, frozenset(), 0)

    def moves(u):
        b, S, p = u
        if b == 0:
            return
        room = len(S) + (1 if p else 0) < m
        sources = set(S) | {0}
        for q in sources:
            if q + 1 <= b and (p or room):
                yield (b, S, q + 1), 1          # (re)use the scratch place for step q + 1
        if p and p + 1 <= b:
            yield (b, S, p + 1), 1              # advance the scratch core by one step
        if p and p not in S:
            yield (b, S | {p}, 0), 0            # commit: the scratch place becomes a stored state
        if p:
            yield (b, S, 0), 0                  # abandon the scratch core
        for q in S:
            yield (b, S - {q}, p), 0            # forget a stored state
        if p == b:
            yield (b - 1, frozenset(q for q in S if q < b), 0), 0
        elif b in S:
            yield (b - 1, S - {b}, p if p < b else 0), 0

    return _zero_one_bfs(start, lambda u: u[0] == 0, moves)


def msm_protocol(t: int, m: int, alpha: int, beta: int | None = None, sigma: int = 1):
    """Cheapest divide-and-conquer tree of the mixed protocol, found by trying them all.

    A tree node handles a subsequence of length n whose start state is stored and chooses
    either a hidden-state push at 1 <= y < n (one unit) or an internal-state push at
    1 <= y <= n (alpha units; beta if y = 1 and the Section 3.4 variant is on; none if y = n,
    because then the state never leaves the working core).  Feasibility is decided by a
    running count of the units in use against the budget m, not by any formula.  ``sigma`` is
    the size of a hidden state in the unit of m (1 in Section 3.3): what a hidden-state push
    takes, and what the start state of the whole sequence occupies from the beginning.
    """
    best = [INFEASIBLE]

    def search(n, in_use, budget_here, spent, cont):
        """Enumerate trees for a subsequence of length n.

        ``in_use`` units are occupied (the start state of this subsequence included);
        ``budget_here`` is what this subtree may reach; ``cont(spent)`` continues with
        whatever remains to be done after the subtree.
        """
        if best[0] is not INFEASIBLE and spent >= best[0]:
            return
        if n == 0:
            cont(spent)
            return
        # hidden-state push at y
        for y in range(1, n):
            if in_use + sigma <= budget_here:
                # right part: starts at the pushed state, may fill the rest of the budget;
                # then the push is released and the left part follows with the full budget
                search(n - y, in_use + sigma, budget_here, spent + y,
                       lambda sp, y=y: search(y, in_use, budget_here, sp, cont))
        # internal-state push at y
        for y in range(1, n + 1):
            if y == n:
                search(y - 1, in_use, budget_here, spent + y, cont)
                continue
            units = beta if (beta is not None and y == 1) else alpha
            # the stored internal state holds the start state of the right part, so the
            # units in use there (its start state included) are in_use + units
            if in_use + units <= budget_here:
                search(n - y, in_use + units, budget_here, spent + y,
                       lambda sp, y=y: search(y - 1, in_use, budget_here, sp, cont))

    def done(spent):
        if best[0] is INFEASIBLE or spent < best[0]:
            best[0] = spent

    if m >= sigma:
        search(t, sigma, m, 0, done)
    return best[0]
