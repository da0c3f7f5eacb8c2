"""The layout simulator against the facts the paper prints about its V-shaped layout (tests/golden/vpp_layout.txt)."""
import os

import pytest

from paper_2608_26523_b200 import schedule as S

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden", "vpp_layout.txt")


def load_golden():
    facts = {}
    with open(GOLDEN) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, val = [x.strip() for x in line.split("=")]
            facts[key] = [int(x) for x in val.split()]
    return facts


def test_stage_placement_and_route():
    g = load_golden()
    lay = S._layout("vpp")
    assert lay["stages"] == g["virtual_stages"][0]
    assert [s for s, r in enumerate(lay["rank_of"]) if r == 0] == g["stages_on_rank0"]
    assert [s for s, r in enumerate(lay["rank_of"]) if r == 1] == g["stages_on_rank1"]
    assert [lay["rank_of"][s] for s in g["route_stages"]] == g["route_ranks"]
    # a chunk's stages depend on one another in route order
    for a, b in zip(g["route_stages"], g["route_stages"][1:]):
        assert (0, 2, a) in S._deps((0, 2, b))


def test_latency_model_and_balance_identity():
    g = load_golden()
    t = 0.75
    tau = S.linear_tau(t)
    assert [tau(k) / t for k in range(len(g["tau_over_t"]))] == pytest.approx(g["tau_over_t"])
    for k in (1, 2, 3):
        exit_prev, entry_next, middle = g["balance_k%d" % k]
        assert tau(k - 1) / t == pytest.approx(exit_prev)
        assert tau(k + 1) / t == pytest.approx(entry_next)
        assert 2 * tau(k) / t == pytest.approx(middle)
        assert exit_prev + entry_next == middle
        assert S.eq3_residual(tau, k) == pytest.approx(0.0, abs=1e-12)
    assert 2 * tau(0) / t == pytest.approx(g["boundary_middle_over_t"][0])
    assert tau(1) / t == pytest.approx(g["boundary_entry_over_t"][0])


def test_rank0_order_and_the_async_swap():
    g = load_golden()
    n = g["example_chunks"][0]
    sync = S.static_orders("vpp", n)[0]
    asyn = S.static_orders("vpp_async", n)[0]
    assert sorted(sync) == sorted(asyn)                    # the same operations ...
    for k in range(1, n - 1):                              # ... with exit of k-1 and entry of k+1 swapped
        exit_prev, entry_next = (0, k - 1, 3), (0, k + 1, 0)
        assert sync.index(exit_prev) + 1 == sync.index(entry_next)
        assert asyn.index(entry_next) + 1 == asyn.index(exit_prev)
    assert g["async_swaps_exit_and_entry"] == [1]
    # rank 1 runs the two middle stages of every chunk back to back, in chunk order
    assert S.static_orders("vpp", n)[1] == [(0, k, s) for k in range(n) for s in g["stages_on_rank1"]]


def test_drain_window_of_the_example():
    g = load_golden()
    n, t = g["example_chunks"][0], 1.5
    for kind in ("vpp", "vpp_async"):
        r = S.simulate(kind, n, S.linear_tau(t))
        assert r.idle[0] / t == pytest.approx(g["drain_over_t"][0])
        assert r.idle[1] / t == pytest.approx(g["drain_over_t"][0])
