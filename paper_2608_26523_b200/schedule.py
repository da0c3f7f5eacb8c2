"""Host-side simulator of the paper's pipeline layouts for chunked prefill on two pipeline ranks (§3.1-3.3):

  CPP        conventional chunked pipeline parallelism: the model is cut in two stages, one per rank
  VPP        four virtual stages folded back over the two ranks (s0, s3 on rank 0; s1, s2 on rank 1), every chunk
             takes the V-shaped route s0 -> s1 -> s2 -> s3, hand-offs are synchronous
  VPP-Async  the same layout with the exit of chunk k-1 and the entry of chunk k+1 swapped on rank 0 so that every
             transfer overlaps computation of the peer
  packing    VPP-Async over a stream of requests: the leading chunks of the next request run in the drain window
             of the current one

It is fed with per-chunk latencies, either the paper's model tau_k = (k + 1) t (Eq. 2) or the latency curve that
bench.py measures for the attention kernel on this GPU (T(P) = a + b P per layer plus a fixed per-layer cost), and
reports makespan, per-rank idle time and the bubble ratio.  Nothing here runs on the GPU and nothing here is on the
attention hot path; it answers "what would the measured cost curve do to the layouts of the paper".

The unit of work is one virtual stage (a quarter of the layers) of one chunk.  A CPP stage is two of them.
"""
from __future__ import annotations

import argparse
import json
from dataclasses import dataclass, field
from typing import Callable, Dict, List, Optional, Sequence, Tuple

Key = Tuple[int, int, int]  # (request, chunk, stage)


@dataclass
class Result:
    start: Dict[Key, float]
    end: Dict[Key, float]
    makespan: float
    busy: List[float]          # compute time per rank
    blocked: List[float]       # time per rank spent inside synchronous transfers
    idle: List[float]          # makespan - busy - blocked
    bubble_ratio: float        # 1 - sum(busy) / (ranks * makespan)
    order: List[List[Key]] = field(default_factory=list)   # what each rank actually ran, in order


def linear_tau(t: float) -> Callable[[int], float]:
    """Eq. 2: per-stage latency of chunk k."""
    return lambda k: (k + 1) * t


def measured_tau(a_ms: float, b_ms_per_token: float, chunk: int, layers_per_stage: int,
                 other_ms_per_layer: float = 0.0) -> Callable[[int], float]:
    """Per-stage latency of chunk k from the measured attention curve T(P) = a + b P (one layer, one chunk of
    `chunk` tokens at prefix P = k * chunk) plus a prefix-independent cost per layer (projections, MoE, norms)."""
    return lambda k: layers_per_stage * (other_ms_per_layer + a_ms + b_ms_per_token * k * chunk)


# ------------------------------------------------------------------------------------------------------------
# layouts: which rank runs a stage, how long it takes, what it depends on, and the static order of each rank
# ------------------------------------------------------------------------------------------------------------
def _layout(kind: str):
    if kind == "cpp":
        return {"stages": 2, "rank_of": [0, 1], "units": [2, 2]}
    if kind in ("vpp", "vpp_async", "packing"):
        return {"stages": 4, "rank_of": [0, 1, 1, 0], "units": [1, 1, 1, 1]}
    raise ValueError("unknown layout %r" % kind)


def static_orders(kind: str, n_chunks: int, req: int = 0) -> List[List[Key]]:
    """The order in which each rank issues its stages for one request (§3.1, §3.2)."""
    if kind == "cpp":
        return [[(req, k, 0) for k in range(n_chunks)], [(req, k, 1) for k in range(n_chunks)]]
    r1 = []
    for k in range(n_chunks):
        r1 += [(req, k, 1), (req, k, 2)]
    r0: List[Key] = [(req, 0, 0)]
    if n_chunks > 1:
        r0.append((req, 1, 0))
    # while rank 1 runs the middle stages of chunk k, rank 0 runs the exit of chunk k-1 and the entry of chunk k+1
    for k in range(1, n_chunks):
        exit_prev, entry_next = (req, k - 1, 3), (req, k + 1, 0)
        pair = [exit_prev, entry_next] if kind == "vpp" else [entry_next, exit_prev]
        r0 += [op for op in pair if op[1] < n_chunks]
    r0.append((req, n_chunks - 1, 3))
    return [r0, r1]


def _deps(key: Key) -> List[Key]:
    req, k, s = key
    d = []
    if s > 0:
        d.append((req, k, s - 1))      # the activation of the same chunk
    if k > 0:
        d.append((req, k - 1, s))      # the prefix KV cache of this stage's layers
    return d


# ------------------------------------------------------------------------------------------------------------
# the simulator
# ------------------------------------------------------------------------------------------------------------
def _finish(start, end, busy, blocked, ran, nranks=2) -> Result:
    makespan = max(end.values()) if end else 0.0
    idle = [makespan - busy[r] - blocked[r] for r in range(nranks)]
    ratio = 1.0 - sum(busy) / (nranks * makespan) if makespan > 0 else 0.0
    return Result(start, end, makespan, busy, blocked, idle, ratio, ran)


def simulate(kind: str, n_chunks: Sequence[int] | int, tau: Callable[[int], float], comm: float = 0.0,
             lookahead: int = 1) -> Result:
    """Run `len(n_chunks)` requests (a single int = one request) through layout `kind`.

    comm is the latency of one cross-rank hand-off; the receiving stage cannot start before it is over.  cpp and vpp
    use synchronous hand-offs: the sender is held for the duration of the transfer as well.  vpp_async and packing
    use asynchronous hand-offs: the sender continues at once.  cpp, vpp and vpp_async run each rank's static order, one request after the other (a request starts when
    the previous one has drained); packing is `simulate_packing`.
    """
    chunks = [n_chunks] if isinstance(n_chunks, int) else list(n_chunks)
    if kind == "packing":
        return simulate_packing(chunks, tau, comm, lookahead)
    lay = _layout(kind)
    rank_of, units = lay["rank_of"], lay["units"]
    nranks = 2
    queues: List[List[Key]] = [[] for _ in range(nranks)]
    for r, n in enumerate(chunks):
        for rk, ops in enumerate(static_orders(kind, n, r)):
            queues[rk] += ops
    sync = kind in ("cpp", "vpp")
    dur = lambda key: units[key[2]] * tau(key[1])
    start: Dict[Key, float] = {}
    end: Dict[Key, float] = {}
    free = [0.0] * nranks              # when the rank can start its next stage
    busy = [0.0] * nranks
    blocked = [0.0] * nranks
    ran: List[List[Key]] = [[] for _ in range(nranks)]
    req_end = [0.0] * len(chunks)
    pos = [0] * nranks
    total = sum(len(q) for q in queues)
    scheduled = 0
    while scheduled < total:
        progressed = False
        for rk in range(nranks):
            if pos[rk] >= len(queues[rk]):
                continue
            key = queues[rk][pos[rk]]
            deps = _deps(key)
            if any(d not in end for d in deps):
                continue
            t = free[rk]
            if key[0] > 0:
                t = max(t, req_end[key[0] - 1])
            for d in deps:
                src = rank_of[d[2]]
                if src == rk:
                    t = max(t, end[d])
                else:
                    t = max(t, end[d] + comm)
            pos[rk] += 1
            start[key] = t
            end[key] = t + dur(key)
            busy[rk] += dur(key)
            free[rk] = end[key]
            if sync and comm > 0.0 and key[2] + 1 < lay["stages"] and rank_of[key[2] + 1] != rk:
                # synchronous send: the sender is held until the hand-off is complete
                free[rk] += comm
                blocked[rk] += comm
            ran[rk].append(key)
            req_end[key[0]] = max(req_end[key[0]], end[key])
            scheduled += 1
            progressed = True
        if not progressed:
            raise RuntimeError("schedule deadlocks: no rank can issue its next stage")
    return _finish(start, end, busy, blocked, ran)


def simulate_packing(chunks: Sequence[int], tau: Callable[[int], float], comm: float = 0.0,
                     lookahead: int = 1) -> Result:
    """VPP-Async over a stream of requests with cross-request packing (§3.3), event-driven.

    Each rank keeps its VPP-Async order over all requests.  Whenever a rank is idle it runs the head of its queue if
    that stage's inputs have arrived; otherwise it may run a later stage of its queue -- at most `lookahead` requests
    ahead of the oldest unfinished one -- whose inputs have arrived and which ends before the head can start (the
    latency model says when: the head's missing input is either on its way or still has to be computed by the peer).
    """
    lay = _layout("packing")
    rank_of, units = lay["rank_of"], lay["units"]
    nranks = 2
    queues: List[List[Key]] = [[] for _ in range(nranks)]
    for r, n in enumerate(chunks):
        for rk, ops in enumerate(static_orders("vpp_async", n, r)):
            queues[rk] += ops
    dur = lambda key: units[key[2]] * tau(key[1])
    start: Dict[Key, float] = {}
    end: Dict[Key, float] = {}
    free = [0.0] * nranks
    busy = [0.0] * nranks
    ran: List[List[Key]] = [[] for _ in range(nranks)]
    left = [list(q) for q in queues]
    remaining = [sum(1 for q in queues for op in q if op[0] == r) for r in range(len(chunks))]

    def arrival(key: Key, rk: int) -> Optional[float]:
        """When all inputs of `key` are on rank rk; None if one of them has not been started yet."""
        t = 0.0
        for d in _deps(key):
            if d not in end:
                return None
            t = max(t, end[d] + (comm if rank_of[d[2]] != rk else 0.0))
        return t

    def earliest(key: Key, rk: int, now: float) -> float:
        """Lower bound on the arrival of `key`'s inputs when some of them have not started: each missing stage takes
        at least its own duration from now on (plus the hand-off if it runs on the peer)."""
        t = now
        for d in _deps(key):
            cross = comm if rank_of[d[2]] != rk else 0.0
            t = max(t, (end[d] if d in end else now + dur(d)) + cross)
        return t

    now = 0.0
    total = sum(len(q) for q in queues)
    scheduled = 0
    guard = 0
    while scheduled < total:
        guard += 1
        if guard > 100 * total + 1000:
            raise RuntimeError("packing simulation does not terminate")
        oldest = min(r for r in range(len(chunks)) if remaining[r] > 0)
        started = False
        for rk in range(nranks):
            if free[rk] > now or not left[rk]:
                continue
            head = left[rk][0]
            ta = arrival(head, rk)
            pick = None
            if ta is not None and ta <= now:
                pick = head
            else:
                th = ta if ta is not None else earliest(head, rk, now)
                for op in left[rk][1:]:
                    if op[0] > oldest + lookahead:
                        break
                    to = arrival(op, rk)
                    if to is not None and to <= now and now + dur(op) <= th:
                        pick = op
                        break
            if pick is None:
                continue
            left[rk].remove(pick)
            start[pick] = now
            end[pick] = now + dur(pick)
            busy[rk] += dur(pick)
            free[rk] = end[pick]
            ran[rk].append(pick)
            remaining[pick[0]] -= 1
            scheduled += 1
            started = True
        if started:
            continue
        # advance to the next event: a rank becomes free or an input arrives
        nxt = [f for f in free if f > now]
        for rk in range(nranks):
            for op in left[rk][:8]:
                ta = arrival(op, rk)
                if ta is not None and ta > now:
                    nxt.append(ta)
        if not nxt:
            raise RuntimeError("packing schedule deadlocks")
        now = min(nxt)
    return _finish(start, end, busy, [0.0] * nranks, ran)


def eq3_residual(tau: Callable[[int], float], k: int) -> float:
    """|tau_{k-1} + tau_{k+1} - 2 tau_k| / (2 tau_k): zero when the latency is affine in k (Eq. 3 holds exactly for the model of Eq. 2)."""
    return abs(tau(k - 1) + tau(k + 1) - 2.0 * tau(k)) / (2.0 * tau(k))


def compare(n_chunks: int, tau: Callable[[int], float], comm: float = 0.0, stream: int = 4) -> Dict[str, dict]:
    """Makespan / bubble ratio of every layout for one request of n_chunks chunks, and of a stream of `stream` such
    requests with and without packing (per-request time = makespan / stream)."""
    out = {}
    for kind in ("cpp", "vpp", "vpp_async"):
        r = simulate(kind, n_chunks, tau, comm)
        out[kind] = {"makespan": r.makespan, "bubble_ratio": r.bubble_ratio, "idle": r.idle, "blocked": r.blocked}
    for kind in ("vpp_async", "packing"):
        r = simulate(kind, [n_chunks] * stream, tau, comm)
        out[kind + "_stream"] = {"makespan": r.makespan, "per_request": r.makespan / stream,
                                 "bubble_ratio": r.bubble_ratio}
    return out


def main(argv=None):
    ap = argparse.ArgumentParser(description=__doc__.split("\n\n")[0])
    ap.add_argument("--bench-json", help="a bench.py output line with a cost_curve (fit_ms a, b_per_token)")
    ap.add_argument("--a-ms", type=float, default=None, help="attention latency at prefix 0, one layer, ms")
    ap.add_argument("--b-ms-per-token", type=float, default=None)
    ap.add_argument("--chunk", type=int, default=8192)
    ap.add_argument("--prompt", type=int, default=131072, help="prompt length in tokens")
    ap.add_argument("--layers", type=int, default=64, help="model layers (a multiple of 4)")
    ap.add_argument("--other-ms", type=float, default=0.0, help="prefix-independent cost per layer and chunk, ms")
    ap.add_argument("--comm-ms", type=float, default=0.0, help="latency of one cross-rank hand-off, ms")
    ap.add_argument("--stream", type=int, default=4)
    args = ap.parse_args(argv)
    a, b = args.a_ms, args.b_ms_per_token
    if args.bench_json:
        line = [l for l in open(args.bench_json) if l.lstrip().startswith("{")][-1]
        d = json.loads(line)
        fit = d["cost_curve"]["fit_ms"]
        a, b = fit["a"], fit["b_per_token"]
        args.chunk = d["config"].get("chunk", args.chunk)
    if a is None or b is None:
        ap.error("give --bench-json or --a-ms and --b-ms-per-token")
    n = (args.prompt + args.chunk - 1) // args.chunk
    tau = measured_tau(a, b, args.chunk, args.layers // 4, args.other_ms)
    res = compare(n, tau, args.comm_ms, args.stream)
    res["inputs"] = {"chunks": n, "chunk": args.chunk, "a_ms": a, "b_ms_per_token": b, "layers": args.layers,
                     "other_ms": args.other_ms, "comm_ms": args.comm_ms,
                     "eq3_residual_mid": eq3_residual(tau, max(1, n // 2))}
    print(json.dumps(res))


if __name__ == "__main__":
    main()
