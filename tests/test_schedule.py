"""Host logic: the pipeline-layout simulator against what the paper's latency model fixes in closed form
(tau_k = (k + 1) t, Eq. 2; tau_{k-1} + tau_{k+1} = 2 tau_k, Eq. 3; drain bubble about (N + 1) t, the pipelined-packing section)."""
import json
import subprocess
import sys

import pytest

from paper_2608_26523_b200 import schedule as S

T = 1.25


def check_valid(res, kind, chunks, tau, comm):
    """Every stage ran exactly once, after its inputs (plus the hand-off when they cross ranks), and a rank never
    runs two stages at once."""
    lay = S._layout(kind)
    nst = lay["stages"]
    want = {(r, k, s) for r, n in enumerate(chunks) for k in range(n) for s in range(nst)}
    assert set(res.start) == want
    for key in want:
        rk = lay["rank_of"][key[2]]
        assert res.end[key] == pytest.approx(res.start[key] + lay["units"][key[2]] * tau(key[1]))
        for d in S._deps(key):
            cross = lay["rank_of"][d[2]] != rk
            assert res.start[key] >= res.end[d] + (comm if cross else 0.0) - 1e-9
    for rk in range(2):
        ops = sorted((res.start[k], res.end[k]) for k in want if lay["rank_of"][k[2]] == rk)
        for (s0, e0), (s1, e1) in zip(ops, ops[1:]):
            assert s1 >= e0 - 1e-9


@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 16])
def test_cpp_closed_form(n):
    # rank 0 never waits: sum 2 tau_k = n (n + 1) t; rank 1 finishes chunk k 2 tau_k after rank 0 -> + 2 n t
    r = S.simulate("cpp", n, S.linear_tau(T))
    assert r.makespan == pytest.approx(n * (n + 1) * T + 2 * n * T)
    assert r.idle[0] == pytest.approx(2 * n * T)          # rank 0 is done 2 tau_{n-1} before the end
    assert r.idle[1] == pytest.approx(2 * n * T)          # 2 t before every chunk
    check_valid(r, "cpp", [n], S.linear_tau(T), 0.0)


@pytest.mark.parametrize("kind", ["vpp", "vpp_async"])
@pytest.mark.parametrize("n", [1, 2, 3, 5, 8, 16])
def test_vpp_closed_form_and_drain_bubble(kind, n):
    # rank 1 works without a gap from t on (Eq. 3: exit of k-1 plus entry of k+1 on rank 0 = the two middle stages
    # of k on rank 1), then rank 0 runs the last exit: t + n (n + 1) t + n t; each rank idles (n + 1) t in total
    r = S.simulate(kind, n, S.linear_tau(T))
    assert r.makespan == pytest.approx(T + n * (n + 1) * T + n * T)
    assert r.idle[0] == pytest.approx((n + 1) * T)
    assert r.idle[1] == pytest.approx((n + 1) * T)
    check_valid(r, kind, [n], S.linear_tau(T), 0.0)


def test_vpp_beats_cpp_for_linear_latency():
    for n in range(2, 20):
        tau = S.linear_tau(T)
        assert S.simulate("vpp", n, tau).makespan < S.simulate("cpp", n, tau).makespan
        assert S.simulate("vpp", n, tau).bubble_ratio < S.simulate("cpp", n, tau).bubble_ratio


def test_eq2_identity_and_residual():
    tau = S.linear_tau(T)
    for k in range(1, 10):
        assert tau(k - 1) + tau(k + 1) == pytest.approx(2 * tau(k))
        assert S.eq3_residual(tau, k) == pytest.approx(0.0, abs=1e-12)
    meas = S.measured_tau(1.1, 0.00024, 8192, 16, other_ms_per_layer=0.3)   # affine in k: the identity still holds
    assert S.eq3_residual(meas, 5) == pytest.approx(0.0, abs=1e-12)
    quad = lambda k: (k + 1) ** 2
    assert S.eq3_residual(quad, 3) == pytest.approx(2.0 / (2 * 16.0))


@pytest.mark.parametrize("comm", [0.1, 0.5, 2.0])
def test_async_hides_handoffs(comm):
    tau = S.linear_tau(T)
    sync = S.simulate("vpp", 8, tau, comm)
    asy = S.simulate("vpp_async", 8, tau, comm)
    check_valid(sync, "vpp", [8], tau, comm)
    check_valid(asy, "vpp_async", [8], tau, comm)
    assert asy.makespan < sync.makespan
    assert sync.blocked[0] == pytest.approx(8 * comm) and sync.blocked[1] == pytest.approx(8 * comm)
    assert asy.blocked == [0.0, 0.0]
    # the route of one chunk crosses ranks twice: no layout can beat the critical path of the last chunk
    assert asy.makespan >= sum(tau(k) for k in range(8)) + 3 * tau(7) + 2 * comm - 1e-9


@pytest.mark.parametrize("n,stream", [(5, 2), (8, 4), (3, 6)])
def test_packing_fills_the_drain_window(n, stream):
    tau = S.linear_tau(T)
    plain = S.simulate("vpp_async", [n] * stream, tau)
    packed = S.simulate("packing", [n] * stream, tau)
    check_valid(packed, "packing", [n] * stream, tau, 0.0)
    assert plain.makespan == pytest.approx(stream * S.simulate("vpp_async", n, tau).makespan)
    assert packed.makespan < plain.makespan
    work = stream * 4 * sum(tau(k) for k in range(n))
    assert packed.makespan >= work / 2 - 1e-9                # two ranks cannot do better than half the work each
    assert packed.bubble_ratio < plain.bubble_ratio


def test_ragged_stream_and_single_chunk_requests():
    tau = S.linear_tau(T)
    chunks = [1, 4, 1, 7, 2]
    for kind in ("cpp", "vpp", "vpp_async", "packing"):
        r = S.simulate(kind, chunks, tau, 0.2)
        check_valid(r, kind, chunks, tau, 0.2)


def test_cli_reads_a_bench_line(tmp_path):
    line = {"config": {"chunk": 8192}, "cost_curve": {"fit_ms": {"a": 1.11, "b_per_token": 0.000234, "r2": 0.9999}}}
    f = tmp_path / "bench.json"
    f.write_text(json.dumps(line) + "\n")
    out = subprocess.run([sys.executable, "-m", "paper_2608_26523_b200.schedule", "--bench-json", str(f), "--prompt",
                          "131072", "--layers", "64", "--comm-ms", "0.5"], capture_output=True, text=True, check=True)
    d = json.loads(out.stdout)
    assert d["inputs"]["chunks"] == 16
    assert d["vpp_async"]["makespan"] < d["vpp"]["makespan"] < d["cpp"]["makespan"]
    assert d["packing_stream"]["per_request"] < d["vpp_async_stream"]["per_request"]
