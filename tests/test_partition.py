"""Pipeline partitioner (paper Section 3.3): the oracle against exhaustive search and closed
cases, then the library's two entry points against the oracle.  Host code only: runs without a GPU."""
import itertools
import math
import time

import numpy as np
import pytest

from oracle import partition_oracle as PO


def _problem(rng, L, D, tight_memory=False, slow_links=False):
    speed = rng.uniform(0.5, 3.0, size=D)
    base = rng.uniform(0.5, 2.0, size=L)
    bw = rng.uniform(0.2, 5.0, size=(D, D)) * (0.05 if slow_links else 10.0)
    return {
        "layers": L, "devices": D,
        "layer_time": (base[None, :] / speed[:, None]).tolist(),
        "out_bytes": rng.uniform(0.5, 2.0, size=L).tolist(),
        "layer_mem": rng.uniform(0.5, 1.5, size=L).tolist(),
        "device_mem": (rng.uniform(1.5, 4.0, size=D) if tight_memory else np.full(D, 1e9)).tolist(),
        "bandwidth": bw.tolist(),
    }


def _compositions(L, k):
    for cuts in itertools.combinations(range(1, L), k - 1):
        b = (0,) + cuts + (L,)
        yield [b[i + 1] - b[i] for i in range(k)]


def _score(problem, comp, devs):
    """Slowest stage of one mapping, evaluated here from the problem's arrays without calling the
    oracle: stage s holds layers [lo, hi) (0-based) on devs[s]; every stage but the last sends the
    output of its last layer, out_bytes[hi - 1], over bandwidth[devs[s]][devs[s + 1]]."""
    lt, ob, lm = problem["layer_time"], problem["out_bytes"], problem["layer_mem"]
    dm, bw = problem["device_mem"], problem["bandwidth"]
    worst, lo = 0.0, 0
    for s, (n, u) in enumerate(zip(comp, devs)):
        hi = lo + n
        if sum(lm[lo:hi]) > dm[u]:
            return math.inf
        worst = max(worst, sum(lt[u][lo:hi]))
        if s + 1 < len(comp):
            worst = max(worst, ob[hi - 1] / bw[u][devs[s + 1]])
        lo = hi
    return worst


def brute_force(problem):
    """Every ordered choice of k distinct devices times every split of L layers into k parts:
    the search space the paper quotes, sum_k D!/(D-k)! * C(L-1, k-1)."""
    L, D = problem["layers"], problem["devices"]
    best, count = math.inf, 0
    for k in range(1, min(L, D) + 1):
        for devs in itertools.permutations(range(D), k):
            for comp in _compositions(L, k):
                count += 1
                best = min(best, _score(problem, comp, devs))
    return best, count


def _args(problem):
    return (problem["layer_time"], problem["out_bytes"], problem["layer_mem"], problem["device_mem"],
            problem["bandwidth"])


# ------------------------------------------------------------------ cases worked by hand
# Each of these has its answer derived in the comment, from Eq. 1-2 alone, and is built so that a
# plausible slip (P_j taken from the wrong layer, b(u,v) read as b(v,u), layer_time indexed
# [layer][device], the last stage charged for sending, a sum where Eq. 2 has a max, "<" for the
# memory check) gives a different T_opt.

def hand_case_asymmetric_links():
    """Two devices, three layers of time 1 and memory 1.  Device 0 holds two layers, device 1 one,
    so exactly two mappings are admissible:
      (a) layers 1-2 on device 0, layer 3 on device 1: T_comp 2 and 1, sends P_2 = 6 over
          b(0,1) = 1 -> T_comm 6 -> period 6
      (b) layer 1 on device 1, layers 2-3 on device 0: T_comp 1 and 2, sends P_1 = 10 over
          b(1,0) = 2 -> T_comm 5 -> period 5
    T_opt = 5 with mapping (b).  P_3 = 1000 is never sent (the last stage sends nothing).
    With b transposed: (a) 3, (b) 10 -> 3.  With P taken one layer late: (a) 1000, (b) 3 -> 3.
    One layer early: (a) 10, (b) 500 or an index error.  Sum instead of max: (b) 2 + 5 = 7.
    Strict memory check: device 0 cannot hold two layers -> infeasible."""
    problem = {"layers": 3, "devices": 2, "layer_time": [[1.0, 1.0, 1.0], [1.0, 1.0, 1.0]],
               "out_bytes": [10.0, 6.0, 1000.0], "layer_mem": [1.0, 1.0, 1.0], "device_mem": [2.0, 1.0],
               "bandwidth": [[777.0, 1.0], [2.0, 555.0]]}
    return problem, 5.0, [(1, 1), (2, 0)]


def hand_case_layer_time_layout():
    """Two devices, four layers, links so fast that T_comm never matters, memory unlimited.
    Device 0 takes [1, 1, 5, 5] per layer, device 1 [4, 4, 1, 1].
      one device:            12 (device 0), 10 (device 1)
      split after layer 1:   0 then 1: max(1, 6) = 6;   1 then 0: max(4, 11) = 11
      split after layer 2:   0 then 1: max(2, 2) = 2;   1 then 0: max(8, 10) = 10
      split after layer 3:   0 then 1: max(7, 1) = 7;   1 then 0: max(9, 5) = 9
    T_opt = 2 with layers 1-2 on device 0 and 3-4 on device 1.  Reading the table as
    [layer][device] (flat index k*D+u) makes both devices [1, 5, 4, 1] and the best split 6."""
    problem = {"layers": 4, "devices": 2, "layer_time": [[1.0, 1.0, 5.0, 5.0], [4.0, 4.0, 1.0, 1.0]],
               "out_bytes": [1.0] * 4, "layer_mem": [1.0] * 4, "device_mem": [1e9, 1e9],
               "bandwidth": [[1e12, 1e12], [1e12, 1e12]]}
    return problem, 2.0, [(2, 0), (2, 1)]


def hand_case_three_devices_link_bound():
    """Three devices, three layers of time 1 everywhere, every device holds one layer, so all
    three are used, one layer each, in some order (6 mappings).  P = [12, 6, 999].
    b(0,1) = 2, b(0,2) = 1, b(1,0) = 4, b(1,2) = 4, b(2,0) = 4, b(2,1) = 6.
    Period = max(1, P_1 / b(first, second), P_2 / b(second, third)):
      0,1,2: max(12/2, 6/4) = 6      0,2,1: max(12/1, 6/6) = 12     1,0,2: max(12/4, 6/1) = 6
      1,2,0: max(12/4, 6/4) = 3      2,0,1: max(12/4, 6/2) = 3      2,1,0: max(12/6, 6/4) = 2
    T_opt = 2 with order 2, 1, 0.  With b transposed the six values are 3, 3, 6, 6, 12, 3 -> 3."""
    bw = [[1.0, 2.0, 1.0], [4.0, 1.0, 4.0], [4.0, 6.0, 1.0]]
    problem = {"layers": 3, "devices": 3, "layer_time": [[1.0] * 3] * 3, "out_bytes": [12.0, 6.0, 999.0],
               "layer_mem": [1.0] * 3, "device_mem": [1.0] * 3, "bandwidth": bw}
    return problem, 2.0, [(1, 2), (1, 1), (1, 0)]


HAND_CASES = [hand_case_asymmetric_links, hand_case_layer_time_layout, hand_case_three_devices_link_bound]


@pytest.mark.parametrize("case", HAND_CASES)
def test_oracle_on_hand_worked_cases(case):
    problem, t_opt, mapping = case()
    for solve in (PO.partition_by_definition, PO.partition):
        got, stages = solve(problem)
        assert got == t_opt                              # exact: the inputs are small integers and halves
        assert stages == mapping
    assert PO.mapping_period(problem, mapping) == t_opt
    assert _score(problem, [n for n, _ in mapping], [u for _, u in mapping]) == t_opt


def test_hand_case_infeasible_with_one_unit_less_memory():
    problem, _, _ = hand_case_asymmetric_links()
    problem["device_mem"] = [1.5, 1.0]                   # three layers of memory 1 no longer fit anywhere
    assert PO.partition_by_definition(problem) == (math.inf, None)
    assert PO.partition(problem) == (math.inf, None)


# ------------------------------------------------------------------ oracle pins
@pytest.mark.parametrize("seed,L,D,tight,slow", [(0, 5, 3, False, False), (1, 6, 4, False, True),
                                                 (2, 6, 3, True, False), (3, 4, 4, True, True),
                                                 (4, 7, 3, False, True), (5, 3, 5, False, False)])
def test_oracle_matches_exhaustive_search(seed, L, D, tight, slow):
    p = _problem(np.random.default_rng(seed), L, D, tight, slow)
    want, count = brute_force(p)
    expect = sum(math.perm(D, k) * math.comb(L - 1, k - 1) for k in range(1, min(L, D) + 1))
    assert count == expect                       # the brute-force search space of Section 3.3
    for solve in (PO.partition_by_definition, PO.partition):
        got, stages = solve(p)
        if math.isinf(want):
            assert stages is None
            continue
        assert got == pytest.approx(want, rel=1e-12)
        assert sum(n for n, _ in stages) == L and len({u for _, u in stages}) == len(stages)
        assert _score(p, [n for n, _ in stages], [u for _, u in stages]) == pytest.approx(got, rel=1e-12)


def test_oracle_homogeneous_devices_fast_links_give_the_most_even_split():
    for L, D in [(12, 4), (12, 5), (7, 3), (4, 8)]:
        p = {"layers": L, "devices": D, "layer_time": [[1.0] * L] * D, "out_bytes": [1.0] * L,
             "layer_mem": [1.0] * L, "device_mem": [1e9] * D, "bandwidth": [[1e12] * D] * D}
        t, stages = PO.partition(p)
        assert t == math.ceil(L / min(L, D))
        assert max(n for n, _ in stages) == math.ceil(L / min(L, D))


def test_oracle_slow_link_and_memory_limit_change_the_answer():
    L, D = 4, 2
    p = {"layers": L, "devices": D, "layer_time": [[1.0] * L] * D, "out_bytes": [10.0] * L,
         "layer_mem": [1.0] * L, "device_mem": [1e9] * D, "bandwidth": [[1.0, 1.0], [1.0, 1.0]]}
    t, stages = PO.partition(p)                  # sending costs 10: one device alone (4) is better
    assert t == 4.0 and len(stages) == 1
    p["device_mem"] = [3.0, 3.0]                 # no device holds all four layers: must split, pays the link
    t, stages = PO.partition(p)
    assert t == 10.0 and len(stages) == 2
    p["device_mem"] = [1.0, 1.0]                 # two devices cannot hold four layers at all
    assert PO.partition(p) == (math.inf, None)


# ------------------------------------------------------------------ library against the oracle
@pytest.fixture(scope="module")
def vit():
    import paper_2110_14895_b200 as v
    from paper_2110_14895_b200 import build as b
    b.build()
    v.lib()
    return v


@pytest.mark.parametrize("case", HAND_CASES)
def test_library_on_hand_worked_cases(vit, case):
    problem, t_opt, mapping = case()
    got, stages = vit.vit_partition(*_args(problem))
    assert got == t_opt and stages == mapping
    # the same problem with every device a category of its own
    got, stages = vit.vit_partition_categories(*_args(problem), [1] * problem["devices"])
    assert got == t_opt and stages == mapping


@pytest.mark.parametrize("seed", range(12))
def test_library_matches_oracle(vit, seed):
    rng = np.random.default_rng(100 + seed)
    L, D = int(rng.integers(2, 10)), int(rng.integers(1, 6))
    p = _problem(rng, L, D, tight_memory=bool(seed % 3 == 0), slow_links=bool(seed % 2))
    want, _ = PO.partition(p)
    if math.isinf(want):
        with pytest.raises(vit.VitError) as e:
            vit.vit_partition(*_args(p))
        assert e.value.status == vit.VIT_ERR_INFEASIBLE
        return
    got, stages = vit.vit_partition(*_args(p))
    assert got == pytest.approx(want, rel=1e-12)
    assert sum(n for n, _ in stages) == L and all(n >= 1 for n, _ in stages)
    assert len({u for _, u in stages}) == len(stages)           # every device at most once
    assert _score(p, [n for n, _ in stages], [u for _, u in stages]) == pytest.approx(got, rel=1e-12)   # the mapping achieves T_opt


def test_library_categories_agree_with_distinct_devices(vit):
    rng = np.random.default_rng(7)
    L, counts = 12, [2, 1, 2]
    N = len(counts)
    cat = _problem(rng, L, N, tight_memory=True)
    cat["device_mem"] = [5.0, 9.0, 3.0]
    owner = [c for c, n in enumerate(counts) for _ in range(n)]
    D = len(owner)
    full = {"layers": L, "devices": D,
            "layer_time": [cat["layer_time"][c] for c in owner], "out_bytes": cat["out_bytes"],
            "layer_mem": cat["layer_mem"], "device_mem": [cat["device_mem"][c] for c in owner],
            "bandwidth": [[cat["bandwidth"][a][b] for b in owner] for a in owner]}
    t_full, _ = vit.vit_partition(*_args(full))
    t_cat, stages = vit.vit_partition_categories(*_args(cat), counts)
    assert t_cat == pytest.approx(t_full, rel=1e-12)
    assert t_cat == pytest.approx(PO.partition(full)[0], rel=1e-12)
    used = [sum(1 for _, c in stages if c == k) for k in range(N)]
    assert all(u <= n for u, n in zip(used, counts)) and sum(n for n, _ in stages) == L


def test_library_argument_errors(vit):
    ok = _problem(np.random.default_rng(0), 4, 2)
    with pytest.raises(vit.VitError) as e:
        big = _problem(np.random.default_rng(0), 4, 17)
        vit.vit_partition(*_args(big))
    assert e.value.status == vit.VIT_ERR_INVALID_ARG
    with pytest.raises(ValueError):
        vit.vit_partition(ok["layer_time"], ok["out_bytes"][:-1], ok["layer_mem"], ok["device_mem"], ok["bandwidth"])
    # values that make no sense are rejected instead of producing a mapping
    for key, idx, bad in (("bandwidth", (0, 1), 0.0), ("bandwidth", (1, 0), -1.0), ("bandwidth", (0, 1), float("nan")),
                          ("layer_time", (1, 2), -0.5), ("layer_time", (0, 0), float("inf")),
                          ("layer_mem", (3,), float("nan")), ("out_bytes", (0,), -1.0), ("device_mem", (1,), float("nan"))):
        p = {k: (np.array(v, dtype=np.float64) if k not in ("layers", "devices") else v) for k, v in ok.items()}
        p[key][idx] = bad
        with pytest.raises(vit.VitError) as e:
            vit.vit_partition(*_args(p))
        assert e.value.status == vit.VIT_ERR_INVALID_ARG, (key, bad)
    with pytest.raises(vit.VitError) as e:
        vit.vit_partition_categories(*_args(ok), [1, -1])
    assert e.value.status == vit.VIT_ERR_INVALID_ARG


def test_table2_configuration_runs_fast(vit):
    """Nine devices in three types of three, a 12-layer model (the configuration of the paper's
    Table 2): the category programme and the subset programme agree; both take well under the
    paper's 0.01 s / 18.6 s."""
    rng = np.random.default_rng(3)
    L, counts = 12, [3, 3, 3]
    cat = _problem(rng, L, 3, tight_memory=True)
    cat["device_mem"] = [2.5, 4.0, 6.0]
    owner = [c for c, n in enumerate(counts) for _ in range(n)]
    full_args = ([cat["layer_time"][c] for c in owner], cat["out_bytes"], cat["layer_mem"],
                 [cat["device_mem"][c] for c in owner], [[cat["bandwidth"][a][b] for b in owner] for a in owner])
    t0 = time.perf_counter(); t_cat, _ = vit.vit_partition_categories(*_args(cat), counts); t1 = time.perf_counter()
    t_full, _ = vit.vit_partition(*full_args); t2 = time.perf_counter()
    assert t_cat == pytest.approx(t_full, rel=1e-12)
    assert t1 - t0 < 0.01 and t2 - t1 < 1.0
