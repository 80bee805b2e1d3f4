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


def brute_force(problem):
    """Every ordered choice of k distinct devices times every split of L layers into k parts:
    the search space the paper quotes, sum_k D!/(D-k)! * C(L-1, k-1)."""
    L, D = problem["layers"], problem["devices"]
    best, count = math.inf, 0
    for k in range(1, min(L, D) + 1):
        for devs in itertools.permutations(range(D), k):
            for comp in _compositions(L, k):
                count += 1
                best = min(best, PO.mapping_period(problem, list(zip(comp, devs))))
    return best, count


def _args(problem):
    return (problem["layer_time"], problem["out_bytes"], problem["layer_mem"], problem["device_mem"],
            problem["bandwidth"])


# ------------------------------------------------------------------ oracle pins
@pytest.mark.parametrize("seed,L,D,tight,slow", [(0, 5, 3, False, False), (1, 6, 4, False, True),
                                                 (2, 6, 3, True, False), (3, 4, 4, True, True),
                                                 (4, 7, 3, False, True), (5, 3, 5, False, False)])
def test_oracle_matches_exhaustive_search(seed, L, D, tight, slow):
    p = _problem(np.random.default_rng(seed), L, D, tight, slow)
    want, count = brute_force(p)
    expect = sum(math.perm(D, k) * math.comb(L - 1, k - 1) for k in range(1, min(L, D) + 1))
    assert count == expect                       # the brute-force search space of Section 3.3
    got, stages = PO.partition(p)
    if math.isinf(want):
        assert stages is None
        return
    assert got == pytest.approx(want, rel=1e-12)
    assert sum(n for n, _ in stages) == L and len({u for _, u in stages}) == len(stages)
    assert PO.mapping_period(p, stages) == pytest.approx(got, rel=1e-12)


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
    assert PO.mapping_period(p, stages) == pytest.approx(got, rel=1e-12)   # the mapping achieves T_opt


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
