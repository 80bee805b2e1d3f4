"""CPU oracle for the pipeline partitioner.  TEST INFRASTRUCTURE ONLY; shares no code with the
library.  Parity status: pinned by hand-worked cases, by closed cases, and -- for the recursion --
by the definition itself on small inputs (tests/test_partition.py).

What is computed (paper Section 3.3).  A mapping is an ordered choice of distinct devices and a
split of the L layers into as many consecutive non-empty parts; it is admissible when every part
fits its device (sum of M_k over the part's layers <= m_u).  Its cost is the slowest stage,
  Eq. 1   T_comm(u, v, P_j) = P_j / b(u, v)
  Eq. 2   T_period = max(T_comp, T_comm)      (computation and communication overlap perfectly)
where a stage that ends with layer j on device u sends P_j to the device v of the next stage, the
last stage sends nothing, and T_comp of a part is the sum of its layers' times on that device.
T_opt is the smallest cost over all admissible mappings.

Two functions compute it:
  * `partition_by_definition`: the minimum written out as a search over every mapping (the
    brute-force space the section quotes).  This is the definition; use it for small inputs.
  * `partition`: the optimal-substructure recurrence of Eq. 3,
        h(j, S + {u}, v) = min over i < j, u not in S of
              max( h(i, S, u), T_comm(u, v, P_j), T_comp({i -> j}, u) ),   h(0, {}, .) = 0,
    evaluated top-down with memoisation (not in the order of the paper's Algorithm 1), for inputs
    the search cannot reach.  Layers are 1-based as in the paper: a part {i -> j} holds layers
    i+1 .. j.
"""
import functools
import itertools
import math


def t_comm(problem, u, v, j):
    """Eq. 1: the output of layer j (1-based) sent from device u to device v."""
    return problem["out_bytes"][j - 1] / problem["bandwidth"][u][v]


def t_comp(problem, i, j, u):
    """Time of layers i+1 .. j (1-based) on device u."""
    return sum(problem["layer_time"][u][k] for k in range(i, j))


def fits(problem, i, j, u):
    """Layers i+1 .. j fit the memory of device u."""
    return sum(problem["layer_mem"][k] for k in range(i, j)) <= problem["device_mem"][u]


def mapping_period(problem, stages):
    """Cost of one mapping [(layer_count, device), ...]: the slowest stage (Eq. 2 per stage);
    inf if a stage does not fit its device."""
    worst, i = 0.0, 0
    for s, (n, u) in enumerate(stages):
        j = i + n
        if not fits(problem, i, j, u):
            return math.inf
        worst = max(worst, t_comp(problem, i, j, u))
        if s + 1 < len(stages):
            worst = max(worst, t_comm(problem, u, stages[s + 1][1], j))
        i = j
    return worst


def all_mappings(L, D):
    """Every ordered choice of k distinct devices times every split of L layers into k parts."""
    for k in range(1, min(L, D) + 1):
        for cuts in itertools.combinations(range(1, L), k - 1):
            bounds = (0,) + cuts + (L,)
            counts = [bounds[s + 1] - bounds[s] for s in range(k)]
            for devs in itertools.permutations(range(D), k):
                yield list(zip(counts, devs))


def partition_by_definition(problem):
    """T_opt as defined: the minimum of `mapping_period` over all mappings.
    Returns (T_opt, one optimal mapping) or (inf, None) when nothing fits."""
    best, arg = math.inf, None
    for stages in all_mappings(problem["layers"], problem["devices"]):
        c = mapping_period(problem, stages)
        if c < best:
            best, arg = c, stages
    return best, arg


def partition(problem):
    """Eq. 3 by memoised recursion.  Returns (T_opt, [(layer_count, device), ...] in pipeline
    order) or (inf, None) when nothing fits."""
    L, D = problem["layers"], problem["devices"]

    @functools.lru_cache(maxsize=None)
    def h(j, used, v):
        """Best slowest-stage time with the first j layers placed on the devices of `used`
        (a frozenset), the next stage going to v (v not in used).  Also returns the (i, u) that
        attains it."""
        if j == 0:
            return (0.0, None) if not used else (math.inf, None)
        best, arg = math.inf, None
        for u in used:
            before = used - {u}
            for i in range(j):
                if not fits(problem, i, j, u):
                    continue
                prev, _ = h(i, before, u)
                c = max(prev, t_comm(problem, u, v, j), t_comp(problem, i, j, u))
                if c < best:
                    best, arg = c, (i, u)
        return best, arg

    # the last stage sends nothing: close the recursion with a stage {i -> L} on u without T_comm
    answer, index = math.inf, None
    for r in range(D):
        for S in itertools.combinations(range(D), r):
            S = frozenset(S)
            for u in range(D):
                if u in S:
                    continue
                for i in range(L):
                    if not fits(problem, i, L, u):
                        continue
                    prev, _ = h(i, S, u)
                    c = max(prev, t_comp(problem, i, L, u))
                    if c < answer:
                        answer, index = c, (i, S, u)
    if index is None:
        return math.inf, None
    i, S, u = index
    stages, j = [], L
    while True:
        stages.append((j - i, u))
        if i == 0:
            break
        _, (pi, pu) = h(i, S, u)
        j, i, u = i, pi, pu
        S = S - {u}
    return answer, stages[::-1]
