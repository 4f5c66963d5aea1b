"""Decode loop over a stack of Virtual-Expert MoE layers with asynchronous expert swapping.

Host-side policy only (SwapMoE Sections 3.1-3.2, Fig. 5 ii): every ``frequency`` steps
the per-layer importance scores (Eq. 1, accumulated on the device by the forward
kernels) are read, the K most important experts are chosen, and the experts that
should enter the resident set are copied from pinned host memory into SPARE arena
entries on a side stream - at most ``loads_per_step`` per layer per step (amortised
loading), never into memory a running forward may read.  A load is committed
``lag`` steps later: the compute stream waits on the copy's event and the slot table
flips to the new arena entry; the evicted entry becomes a spare.  Until the flip
the old expert keeps serving the slot.

Readings where the paper is silent: entering experts are taken in descending
importance, victims are the least important residents that left the top-K, and the
importance window is reset at every decision.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import List, Optional, Sequence

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
    queue: List[tuple] = field(default_factory=list)       # (expert_in, slot) waiting for a spare entry
    pending: List[_Pending] = field(default_factory=list)  # copies in flight / awaiting commit


class DecodeStack:
    """L independent layers driven step by step; records the slot tables each step used."""

    def __init__(self, layers: Sequence[LayerState], frequency: int = 8, loads_per_step: int = 1,
                 lag: int = 2, compute_stream=None, side_stream=None, time_loads: bool = False,
                 graph_buffers=None):
        import torch
        self.layers = list(layers)
        self.frequency, self.loads_per_step, self.lag = int(frequency), int(loads_per_step), int(lag)
        self.compute = compute_stream or torch.cuda.current_stream()
        self.side = side_stream or torch.cuda.Stream()
        self.step_no = 0
        self.trace = []            # (step, layer, s2e copy, phys copy)
        self.decisions = []        # (step, layer, importance read, top-K chosen)
        self.stalls = 0            # commits whose copy had not finished when the flip was enqueued
        self.loads = 0
        self.bytes_loaded = 0
        self.time_loads = time_loads
        self.load_events = []      # (start, stop) events around every copy when time_loads is set
        # graph_buffers = (x_buf, out_buf), device tensors [L, B, d_model]: the L forwards of a step
        # are then captured once into a CUDA graph over these fixed buffers and replayed
        # (step_graph); slot-table flips and expert copies stay outside the graph.
        self.graph_buffers = graph_buffers
        self.graph = None
        for st in self.layers:
            st.layer.set_resident(st.s2e, st.arena_in, st.arena_out, st.phys, stream=self.compute)

    # ---------------------------------------------------------------- one step
    def step(self, xs: Sequence, outs: Sequence, record: bool = True) -> None:
        """xs[l], outs[l]: device tensors [B, d_model] of layer l for this step."""
        n = self.step_no
        for li, st in enumerate(self.layers):
            self._commit_due(st, n)
            if record:
                self.trace.append((n, li, st.s2e.copy(), st.phys.copy()))
            st.layer.forward(xs[li], outs[li], stream=self.compute)
        if (n + 1) % self.frequency == 0:
            for li, st in enumerate(self.layers):
                self._decide(li, st, n)
        for st in self.layers:
            self._issue_loads(st, n)
        self.step_no += 1

    def step_graph(self, x_step, record: bool = False) -> None:
        """One step through the captured graph: x_step [L, B, d_model] is copied into the fixed
        input buffer, due table flips are enqueued, the graph runs, the scheduler acts."""
        import torch
        x_buf, out_buf = self.graph_buffers
        n = self.step_no
        with torch.cuda.stream(self.compute):
            if self.graph is None:
                for li, st in enumerate(self.layers):          # eager once: lazily built state
                    st.layer.forward(x_buf[li], out_buf[li], stream=self.compute)
                    st.layer.read_importance(reset=True, stream=self.compute)
                self.compute.synchronize()
                self.graph = torch.cuda.CUDAGraph()
                with torch.cuda.graph(self.graph, capture_error_mode="thread_local"):   # torch's own side stream
                    for li, st in enumerate(self.layers):
                        st.layer.forward(x_buf[li], out_buf[li], stream=None)
            x_buf.copy_(x_step, non_blocking=True)
            for li, st in enumerate(self.layers):
                self._commit_due(st, n)
                if record:
                    self.trace.append((n, li, st.s2e.copy(), st.phys.copy()))
            self.graph.replay()
        if (n + 1) % self.frequency == 0:
            for li, st in enumerate(self.layers):
                self._decide(li, st, n)
        for st in self.layers:
            self._issue_loads(st, n)
        self.step_no += 1

    def loader_seconds(self) -> float:
        """Sum of the device-side durations of all copies issued so far (needs time_loads)."""
        return sum(a.elapsed_time(b) for a, b in self.load_events) * 1e-3

    def _commit_due(self, st: LayerState, n: int) -> None:
        due = [p for p in st.pending if p.commit_step <= n]
        if not due:
            return
        for p in due:
            if not p.event.query():
                self.stalls += 1
            self.compute.wait_event(p.event)
            old = int(st.phys[p.slot])
            st.s2e[p.slot] = p.expert
            st.phys[p.slot] = p.phys
            st.spare.append(old)
            st.pending.remove(p)
        st.layer.set_resident(st.s2e, st.arena_in, st.arena_out, st.phys, stream=self.compute)

    def _decide(self, li: int, st: LayerState, n: int) -> None:
        K = st.layer.cfg.K
        imp = st.layer.read_importance(reset=True, stream=self.compute)
        top = binding.topk_importance(imp, K)
        self.decisions.append((n, li, imp.copy(), top.copy()))
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

    def _issue_loads(self, st: LayerState, n: int) -> None:
        import torch
        issued = 0
        while st.queue and st.spare and issued < self.loads_per_step:
            expert, slot = st.queue.pop(0)
            phys = st.spare.pop(0)
            ev = torch.cuda.Event()
            # the spare entry may still be read by forwards already enqueued before its slot
            # was flipped away: order the copy after everything enqueued so far
            self.side.wait_stream(self.compute)
            if self.time_loads:
                t0 = torch.cuda.Event(enable_timing=True)
                ev = torch.cuda.Event(enable_timing=True)
                t0.record(self.side)
                self.load_events.append((t0, ev))
            st.layer.load_slot_async(phys, st.host_in[expert], st.host_out[expert], self.side, ev)
            st.pending.append(_Pending(n + self.lag, slot, expert, phys, ev))
            issued += 1
            self.loads += 1
            self.bytes_loaded += st.host_in[expert].numel() * st.host_in.element_size() + \
                st.host_out[expert].numel() * st.host_out.element_size()
