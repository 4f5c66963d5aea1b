"""Decode loop over a stack of Virtual-Expert MoE layers with asynchronous expert swapping.

Host-side policy only (SwapMoE Sections 3.1-3.2, Fig. 5 ii): every ``frequency`` steps
the per-layer importance scores (Eq. 1, accumulated on the device by the forward
kernels) are read, the K most important experts are chosen, and the experts that
should enter the resident set are copied from pinned host memory into SPARE arena
entries on a side stream (amortised loading: at most ``loads_per_step`` per layer and
``step_budget`` over all layers per step), never into memory a running forward may
read.  A load becomes eligible for its commit ``lag`` steps later.  With
``commit="wait"`` the compute stream then waits on the copy's event and the slot
table flips (deterministic schedule; a wait that actually blocks is counted as a
stall).  With ``commit="ready"`` the table flips only if the copy HAS finished
(event query); otherwise the old expert keeps serving the slot and the commit is
retried at the next step, so loading never blocks inference.  Every step's tables
are recorded in ``trace`` either way, so a replay of the trace is exact.  The
evicted entry becomes a spare.

Each layer object carries its own resident budget K (the configuration tuple
{frequency, #experts_1..L} of Section 3.3): the layers of a stack may differ in K.

Two comparison policies of Section 4.1 run over the same kernels:
``policy="static_pruning"`` keeps the K experts with the largest ||E_i|| and never
updates; ``policy="on_demand"`` loads a requested expert that is not resident
synchronously (the compute stream waits for the copy) and runs the layer again.

Readings where the paper is silent: entering experts are taken in descending
importance, victims are the least important residents that left the top-K, and the
importance window is reset at every decision.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Callable, List, Optional, Sequence

import numpy as np

from . import binding


@dataclass
class _Pending:
    commit_step: int
    slot: int
    expert: int
    phys: int
    event: object


@dataclass
class LayerState:
    layer: binding.Layer
    s2e: np.ndarray              # [K] expert served by each logical slot
    phys: np.ndarray             # [K] arena entry backing each logical slot
    spare: List[int]             # arena entries no slot points at
    arena_in: object             # device [K+S, nin, f, d]
    arena_out: object            # device [K+S, d, f]
    host_in: object              # pinned [E, nin, f, d]
    host_out: object             # pinned [E, d, f]
    enorm: Optional[np.ndarray] = None                     # [E] ||E_i|| (static_pruning picks by it)
    queue: List[tuple] = field(default_factory=list)       # (expert_in, slot) waiting for a spare entry
    pending: List[_Pending] = field(default_factory=list)  # copies in flight / awaiting commit
    last_used: Optional[np.ndarray] = None                 # [K] step at which each slot last served a token (on_demand)


def suggest_step_budget(step_seconds: float, pcie_gbytes_per_s: float, expert_bytes: int, share: float = 0.9) -> float:
    """Loads per step that the host link can carry while a step runs (Section 3.4.1: the update
    traffic must stay below what the link delivers in the time the computation takes).  May be a
    fraction: 0.5 means one load every other step."""
    return share * step_seconds * pcie_gbytes_per_s * 1e9 / expert_bytes


class DecodeStack:
    """L independent layers driven step by step; records the slot tables each step used."""

    def __init__(self, layers: Sequence[LayerState], frequency: int = 8, loads_per_step: int = 1,
                 lag: int = 2, compute_stream=None, side_stream=None, time_loads: bool = False,
                 graph_buffers=None, step_budget: Optional[float] = None, commit: str = "wait",
                 policy: str = "swap", event_factory: Optional[Callable[[], object]] = None,
                 track_hits: bool = False, async_decide: bool = False,
                 score_alloc: Optional[Callable[[int], object]] = None, max_in_flight: Optional[int] = None):
        import torch
        assert commit in ("wait", "ready") and policy in ("swap", "static_pruning", "on_demand")
        self.layers = list(layers)
        self.frequency, self.loads_per_step, self.lag = int(frequency), int(loads_per_step), int(lag)
        # step_budget: loads per step over all layers; fractions accumulate from step to step (0.5 = one
        # load every other step), whole budgets do not carry over
        self.step_budget = None if step_budget is None else float(step_budget)
        self._bucket = 0.0
        self.commit, self.policy = commit, policy
        self.compute = compute_stream or torch.cuda.current_stream()
        self.side = side_stream or torch.cuda.Stream()
        self.new_event = event_factory or (lambda: torch.cuda.Event(enable_timing=self.time_loads))
        self.step_no = 0
        self.trace = []            # (step, layer, s2e copy, phys copy)
        self.decisions = []        # (step, layer, importance read, top-K chosen)
        self.stalls = 0            # commit="wait": commits whose copy had not finished when the flip was enqueued
        self.deferred = 0          # commit="ready": commits put off to a later step because the copy was still running
        self.commits = 0
        self.loads = 0
        self.bytes_loaded = 0
        self.misses = 0            # on_demand: requested experts that were not resident
        self.blocking_loads = 0    # on_demand: loads the compute stream waited for
        self.requests = 0          # on_demand: (token, expert) requests seen
        # async_decide: the scores of a decision step are only ENQUEUED for copy-out (pinned buffers, one event);
        # the top-K choice is made at a later step, once the event has fired - the host never waits for the
        # device, so the queue of forwards never drains
        # max_in_flight: the host enqueues step n only once step n - max_in_flight has finished on the device (an
        # autoregressive decoder cannot run further ahead than its sampler anyway).  Without a bound a host that
        # is faster than the device queues hundreds of steps, every expert copy - ordered behind the queue - lands
        # that much later, and the resident sets lag behind the traffic they are meant to follow.
        self.max_in_flight = max_in_flight
        self._step_events = []
        self.host_seconds = 0.0    # host time spent preparing and enqueuing steps (waits for the device excluded)
        self.throttle_waits = 0    # steps before which the host had to wait for the device (max_in_flight)
        self._t_step = None
        self.async_decide = async_decide
        self.score_alloc = score_alloc or (lambda E: torch.empty((3, E), dtype=torch.float32).pin_memory())
        self._inflight = None      # (step, event, [pinned score tensors per layer]) of the decision being read
        self._todo = []            # layers of that decision still to be decided
        self.decisions_per_step = max(1, -(-len(self.layers) // max(1, min(4, self.frequency - 1))))
        self.track_hits = track_hits
        self.hits = 0              # track_hits: requests of the off-the-shelf gate that met a resident expert ...
        self.asked = 0             # ... out of this many (read at every decision; the table at the decision counts)
        self.time_loads = time_loads
        self.load_events = []      # (start, stop) events around every copy when time_loads is set
        # graph_buffers = (x_buf, out_buf), device tensors [L, B, d_model]: the L forwards of a step
        # are then captured once into a CUDA graph over these fixed buffers and replayed
        # (step_graph); slot-table flips and expert copies stay outside the graph.
        self.graph_buffers = graph_buffers
        self.graph = None
        self.graph_launches = 0          # library kernels in the captured step
        self.graph_replays = 0
        for st in self.layers:
            st.layer.set_resident(st.s2e, st.arena_in, st.arena_out, st.phys, stream=self.compute)
            st.last_used = np.zeros(st.layer.cfg.K, np.int64)
        if policy == "static_pruning":
            for st in self.layers:
                self._install_pruning_set(st)

    # ---------------------------------------------------------------- one step
    def step(self, xs: Sequence, outs: Sequence, record: bool = True) -> None:
        """xs[l], outs[l]: device tensors [B, d_model] of layer l for this step."""
        n = self.step_no
        self._throttle()
        for li, st in enumerate(self.layers):
            self._commit_due(st, n)
            if self.policy == "on_demand":
                self._forward_on_demand(li, st, xs[li], outs[li], n, record)
                continue
            if record:
                self.trace.append((n, li, st.s2e.copy(), st.phys.copy()))
            st.layer.forward(xs[li], outs[li], stream=self.compute)
        self._mark_step()
        self._schedule(n)
        self.step_no += 1

    def step_graph(self, x_step, record: bool = False) -> None:
        """One step through the captured graph: x_step [L, B, d_model] is copied into the fixed
        input buffer, due table flips are enqueued, the graph runs, the scheduler acts."""
        import torch
        assert self.policy != "on_demand", "on-demand loading decides inside the step: use step()"
        x_buf, out_buf = self.graph_buffers
        n = self.step_no
        with torch.cuda.stream(self.compute):
            if self.graph is None:
                for li, st in enumerate(self.layers):          # eager once: lazily built state
                    st.layer.forward(x_buf[li], out_buf[li], stream=self.compute)
                    st.layer.read_importance(reset=True, stream=self.compute)
                self.compute.synchronize()
                self.graph = torch.cuda.CUDAGraph()
                l0 = sum(st.layer.launch_count for st in self.layers)
                with torch.cuda.graph(self.graph, capture_error_mode="thread_local"):   # torch's own side stream
                    for li, st in enumerate(self.layers):
                        st.layer.forward(x_buf[li], out_buf[li], stream=None)
                self.graph_launches = sum(st.layer.launch_count for st in self.layers) - l0   # kernels per replay
            self._throttle()
            x_buf.copy_(x_step, non_blocking=True)
            for li, st in enumerate(self.layers):
                self._commit_due(st, n)
                if record:
                    self.trace.append((n, li, st.s2e.copy(), st.phys.copy()))
            self.graph.replay()
            self.graph_replays += 1
            self._mark_step()
        self._schedule(n)
        self.step_no += 1

    def _throttle(self) -> None:
        import time
        t0 = time.perf_counter()
        if self._t_step is not None:
            self.host_seconds += t0 - self._t_step       # host work of the step before (everything but this wait)
        if self.max_in_flight is not None and len(self._step_events) >= self.max_in_flight:
            ev = self._step_events.pop(0)
            if not ev.query():
                ev.synchronize()
                self.throttle_waits += 1                   # the device was still busy: the host is ahead
        self._t_step = time.perf_counter()

    def _mark_step(self) -> None:
        if self.max_in_flight is not None:
            ev = self.new_event()
            ev.record(self.compute)
            self._step_events.append(ev)

    def loader_seconds(self) -> float:
        """Sum of the device-side durations of all copies issued so far (needs time_loads)."""
        return sum(a.elapsed_time(b) for a, b in self.load_events) * 1e-3

    # ---------------------------------------------------------------- scheduler (Sections 3.1-3.2)
    def _schedule(self, n: int) -> None:
        if self.policy != "swap":
            return
        if self.async_decide:
            self._decide_async(n)
        elif (n + 1) % self.frequency == 0:
            for li, st in enumerate(self.layers):
                self._decide(li, st, n)
        # amortised loading: the step's budget is dealt round-robin, starting at a layer that
        # moves on every step so that no layer's queue is starved
        L = len(self.layers)
        if self.step_budget is not None:
            self._bucket = min(self._bucket + self.step_budget, max(1.0, self.step_budget))
            left = int(self._bucket + 1e-9)
        else:
            left = L * self.loads_per_step
        issued = [0] * L
        progress = True
        while left > 0 and progress:
            progress = False
            for i in range(L):
                li = (n + i) % L
                st = self.layers[li]
                if left > 0 and issued[li] < self.loads_per_step and st.queue and st.spare:
                    self._issue_load(st, n)
                    issued[li] += 1
                    left -= 1
                    self._bucket -= 1.0
                    progress = True

    def _commit_due(self, st: LayerState, n: int) -> None:
        due = [p for p in st.pending if p.commit_step <= n]
        if not due:
            return
        flipped = False
        for p in due:
            if not p.event.query():
                if self.commit == "ready":
                    self.deferred += 1          # the old expert keeps serving; try again next step
                    continue
                self.stalls += 1
            if self.commit == "wait":
                self.compute.wait_event(p.event)
            old = int(st.phys[p.slot])
            st.s2e[p.slot] = p.expert
            st.phys[p.slot] = p.phys
            st.spare.append(old)
            st.pending.remove(p)
            self.commits += 1
            flipped = True
        if flipped:
            st.layer.set_resident(st.s2e, st.arena_in, st.arena_out, st.phys, stream=self.compute)

    def _decide_async(self, n: int) -> None:
        if self._inflight is not None and (self._todo or self._inflight[1].query()):
            # the scores have landed: the layers' decisions are taken a few per step, so that no step has to
            # wait for the host to work through all of them (the device only has max_in_flight steps queued)
            n0, _, bufs = self._inflight
            if not self._todo:
                self._todo = list(range(len(self.layers)))
            for li in [self._todo.pop(0) for _ in range(min(len(self._todo), self.decisions_per_step))]:
                st = self.layers[li]
                E = st.layer.cfg.E
                self._decide(li, st, n0, imp=bufs[li][0, :E].numpy().copy(),
                             cnt=bufs[li][1, :E].numpy().copy() if self.track_hits else None)
            if not self._todo:
                self._inflight = None
        if (n + 1) % self.frequency == 0 and self._inflight is None:
            if not hasattr(self, "_score_bufs"):
                self._score_bufs = [self.score_alloc(st.layer.cfg.E) for st in self.layers]
            kinds = ("eq1", "count") if self.track_hits else ("eq1",)
            for li, st in enumerate(self.layers):
                st.layer.read_scores_async(kinds, self._score_bufs[li], reset=True, stream=self.compute)
            ev = self.new_event()
            ev.record(self.compute)
            self._inflight = (n, ev, self._score_bufs)

    def _decide(self, li: int, st: LayerState, n: int, imp=None, cnt=None) -> None:
        K = st.layer.cfg.K
        if imp is None:
            imp = st.layer.read_importance(reset=True, stream=self.compute)
            if self.track_hits:
                cnt = st.layer.read_score("count", reset=True, stream=self.compute)
        top = binding.topk_importance(imp, K)
        self.decisions.append((n, li, imp.copy(), top.copy()))
        if cnt is not None:
            self.hits += float(cnt[st.s2e].sum())
            self.asked += float(cnt.sum())
        # residents after all pending commits
        future = st.s2e.copy()
        for p in st.pending:
            future[p.slot] = p.expert
        resident = set(int(e) for e in future)
        want = [int(e) for e in top if int(e) not in resident]                 # descending importance
        keep = set(int(e) for e in top)
        busy = set(p.slot for p in st.pending)
        victims = sorted((s for s in range(K) if int(future[s]) not in keep and s not in busy),
                         key=lambda s: (imp[int(future[s])], int(future[s])))  # least important first
        st.queue = list(zip(want, victims))

    def _issue_load(self, st: LayerState, n: int, expert: Optional[int] = None, slot: Optional[int] = None):
        import torch
        if expert is None:
            expert, slot = st.queue.pop(0)
        phys = st.spare.pop(0)
        ev = self.new_event()
        if self.time_loads:
            # the copy is ordered behind the compute stream by the library; the start event has to sit
            # behind that wait too, or it would time the wait
            t0 = torch.cuda.Event(enable_timing=True)
            self.side.wait_stream(self.compute)
            t0.record(self.side)
            self.load_events.append((t0, ev))
        # the spare entry may still be read by forwards enqueued before its slot was flipped away:
        # the library orders the copy behind everything enqueued so far on the compute stream
        st.layer.load_slot_async(phys, st.host_in[expert], st.host_out[expert], self.compute, self.side, ev)
        p = _Pending(n + self.lag, slot, expert, phys, ev)
        st.pending.append(p)
        self.loads += 1
        if li_bytes := getattr(st, "_expert_bytes", None):
            self.bytes_loaded += li_bytes
        else:
            st._expert_bytes = st.host_in[expert].numel() * st.host_in.element_size() + \
                st.host_out[expert].numel() * st.host_out.element_size()
            self.bytes_loaded += st._expert_bytes
        return p

    # ---------------------------------------------------------------- comparison policies (Section 4.1)
    def _install_pruning_set(self, st: LayerState) -> None:
        """"Pruning": the K experts with the largest ||E_i|| become resident once, for good."""
        assert st.enorm is not None, "static_pruning needs LayerState.enorm"
        K = st.layer.cfg.K
        target = [int(e) for e in binding.topk_importance(np.asarray(st.enorm, np.float32), K)]
        have = set(int(e) for e in st.s2e)
        slots = [s for s in range(K) if int(st.s2e[s]) not in target]
        for e in (e for e in target if e not in have):
            p = self._issue_load(st, -1, expert=e, slot=slots.pop(0))
            p.commit_step = -1
            self.compute.wait_event(p.event)
            self._flip(st, p)         # the library must know the new table before the freed entry is loaded into
            st.layer.set_resident(st.s2e, st.arena_in, st.arena_out, st.phys, stream=self.compute)

    def _flip(self, st: LayerState, p: _Pending) -> None:
        old = int(st.phys[p.slot])
        st.s2e[p.slot] = p.expert
        st.phys[p.slot] = p.phys
        st.spare.append(old)
        st.pending.remove(p)
        self.commits += 1

    def _forward_on_demand(self, li: int, st: LayerState, x, out, n: int, record: bool) -> None:
        """"On demand": run the layer, look at which experts the off-the-shelf gate asked for, and if
        one of them is not resident load it now - the compute stream waits for the copy - and run
        the layer again.  Victims are the slots unused for the longest time that this step does not
        want; with more distinct requests than slots the most requested experts win."""
        K = st.layer.cfg.K
        st.layer.forward(x, out, stream=self.compute)
        uidx = st.layer.tap("uidx", stream=self.compute).reshape(-1)       # host sync: the policy is synchronous
        self.requests += uidx.size
        ids, cnt = np.unique(uidx, return_counts=True)
        wanted = [int(e) for e in ids[np.argsort(-cnt, kind="stable")]][:K]
        resident = {int(e): s for s, e in enumerate(st.s2e)}
        missing = [e for e in wanted if e not in resident]
        self.misses += int(sum(cnt[list(ids).index(e)] for e in missing))
        for e in wanted:
            if e in resident:
                st.last_used[resident[e]] = n + 1
        if missing:
            free = sorted((s for s in range(K) if int(st.s2e[s]) not in wanted), key=lambda s: (st.last_used[s], s))
            for e in missing:
                if not free or not st.spare:
                    break
                p = self._issue_load(st, n, expert=e, slot=free.pop(0))
                self.compute.wait_event(p.event)                           # the load blocks inference
                self.blocking_loads += 1
                st.last_used[p.slot] = n + 1
                self._flip(st, p)
                st.layer.set_resident(st.s2e, st.arena_in, st.arena_out, st.phys, stream=self.compute)
            st.layer.forward(x, out, stream=self.compute)
        if record:
            self.trace.append((n, li, st.s2e.copy(), st.phys.copy()))
