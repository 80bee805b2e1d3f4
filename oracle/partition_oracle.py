"""CPU oracle for the pipeline partitioner.  TEST INFRASTRUCTURE ONLY; shares no code with the
library.  Parity status: pinned by exhaustive search on small inputs and by closed cases
(tests/test_partition.py).

What is computed (paper Section 3.3):
  Eq. 1   T_comm(u, v, P_j) = P_j / b(u, v)
  Eq. 2   T_period = max(T_comp, T_comm): computation and communication overlap perfectly
  Eq. 3   h(j, S + {u}, v) = min over i < j, u not in S of
              max( h(i, S, u), T_comm(u, v, P_j), T_comp({i -> j}, u) ),   h(0, {}, .) = 0
  Algorithm 1: the memoised evaluation with the memory check (sum of M_k over the stage's layers
  must not exceed m_u), the last stage sending nothing, and a precursor table for the mapping.
T_comp of a layer range is the sum of the per-layer times on that device.
"""
import itertools
import math


def t_comm(problem, u, v, j):
    """Eq. 1 for a stage that ends with layer j (1-based)."""
    return problem["out_bytes"][j - 1] / problem["bandwidth"][u][v]


def t_comp(problem, i, j, u):
    """Time of layers i+1 .. j (1-based) on device u."""
    return sum(problem["layer_time"][u][k] for k in range(i, j))


def fits(problem, i, j, u):
    return sum(problem["layer_mem"][k] for k in range(i, j)) <= problem["device_mem"][u]


def partition(problem):
    """Algorithm 1.  Returns (T_opt, [(layer_count, device), ...] in pipeline order) or
    (inf, None) when nothing fits."""
    L, D = problem["layers"], problem["devices"]
    h = {(0, frozenset(), u): 0.0 for u in range(D)}
    precursor = {}
    answer, index = math.inf, None
    subsets = [frozenset(c) for r in range(D + 1) for c in itertools.combinations(range(D), r)]
    for i in range(L):
        for S in subsets:
            for u in range(D):
                if u in S or (i, S, u) not in h:
                    continue
                for j in range(i + 1, L + 1):
                    if not fits(problem, i, j, u):
                        break
                    if j == L:
                        C = max(h[(i, S, u)], t_comp(problem, i, j, u))
                        if C < answer:
                            answer, index = C, (i, S, u)
                    else:
                        S2 = S | {u}
                        for v in range(D):
                            if v in S2:
                                continue
                            C = max(h[(i, S, u)], t_comm(problem, u, v, j), t_comp(problem, i, j, u))
                            if C < h.get((j, S2, v), math.inf):
                                h[(j, S2, v)] = C
                                precursor[(j, S2, v)] = (i, u)
    if index is None:
        return math.inf, None
    i, S, u = index
    stages, j = [], L
    while True:
        stages.append((j - i, u))
        if i == 0:
            break
        pi, pu = precursor[(i, S, u)]
        j, i, u = i, pi, pu
        S = S - {u}
    return answer, stages[::-1]


def mapping_period(problem, stages):
    """The slowest stage of a given mapping [(layer_count, device)]: max over stages of
    max(T_comp, T_comm to the next stage); inf if a stage does not fit its device."""
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
