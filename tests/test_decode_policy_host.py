"""Host-side logic of the decode loop's scheduler, with fakes for the layer, the streams and the
copy events (no GPU): asynchronous loading must not block inference (Section 3.2, Fig. 5 ii), the
per-step load budget is honoured and dealt fairly (amortised loading), and the step budget follows
the link rate (Section 3.4.1)."""
import numpy as np
import torch

from paper_2308_15030_b200 import binding
from paper_2308_15030_b200.decode import DecodeStack, LayerState, suggest_step_budget


class FakeEvent:
    def __init__(self):
        self.done = False

    def query(self):
        return self.done

    def record(self, stream):
        pass


class FakeStream:
    def __init__(self):
        self.waited = []

    def wait_event(self, ev):
        self.waited.append(ev)

    def wait_stream(self, other):
        pass


class FakeCfg:
    def __init__(self, K, E):
        self.K, self.E = K, E


class FakeLayer:
    """Stands in for binding.Layer: records tables and forwards, serves a scripted importance."""

    def __init__(self, K, E):
        self.cfg = FakeCfg(K, E)
        self.tables, self.forwards, self.loads = [], [], []
        self.imp = np.zeros(E, np.float32)

    def set_resident(self, s2e, a_in, a_out, phys, stream=None):
        self.tables.append((np.array(s2e).copy(), np.array(phys).copy()))

    def forward(self, x, out, stream=None):
        self.forwards.append(self.tables[-1][0].copy())

    def read_importance(self, reset=False, stream=None):
        return self.imp.copy()

    def load_slot_async(self, phys, h_in, h_out, compute, side, ev):
        self.loads.append((phys, ev))

    def read_scores_async(self, kinds, out, reset=False, stream=None):
        out[0, : self.cfg.E] = torch.from_numpy(self.imp)


class FakeHost:
    """Indexable like a pinned tensor bank; every expert is 8 bytes."""

    def __getitem__(self, e):
        return self

    def numel(self):
        return 4

    def element_size(self):
        return 1


def _stack(n_layers=1, K=2, E=6, spare=1, **kw):
    # binding.topk_importance is a pure host function of the library (no GPU needed)
    layers = [LayerState(FakeLayer(K, E), np.arange(K, dtype=np.int32), np.arange(K, dtype=np.int32),
                         list(range(K, K + spare)), None, None, FakeHost(), FakeHost()) for _ in range(n_layers)]
    comp, side = FakeStream(), FakeStream()
    st = DecodeStack(layers, compute_stream=comp, side_stream=side, event_factory=FakeEvent, **kw)
    return st, layers, comp


def test_withheld_copy_never_blocks_and_old_slot_keeps_serving():
    stack, layers, comp = _stack(frequency=1, lag=1, commit="ready")
    L = layers[0].layer
    L.imp[:] = [1, 1, 9, 0, 0, 0]                    # expert 2 should enter, one of 0/1 leaves
    for _ in range(6):
        stack.step([None], [None])
    # one load was issued; its completion is withheld: the table never flipped, nobody waited
    assert len(L.loads) == 1 and stack.loads == 1
    assert comp.waited == []
    assert all(np.array_equal(t, [0, 1]) for t in L.forwards)
    assert all(np.array_equal(tr[2], [0, 1]) for tr in stack.trace)
    assert stack.deferred >= 4 and stack.commits == 0 and stack.stalls == 0
    # the copy lands: the next step flips, still without a wait, and the evicted entry is spare again
    L.loads[0][1].done = True
    stack.step([None], [None])
    assert comp.waited == []
    assert 2 in L.forwards[-1].tolist() and stack.commits == 1
    assert sorted(stack.trace[-1][3].tolist() + layers[0].spare) == [0, 1, 2]


def test_wait_mode_orders_the_compute_stream_behind_the_copy_and_counts_the_stall():
    stack, layers, comp = _stack(frequency=1, lag=1, commit="wait")
    L = layers[0].layer
    L.imp[:] = [1, 1, 9, 0, 0, 0]
    for _ in range(3):
        stack.step([None], [None])
    assert len(comp.waited) == 1 and stack.stalls == 1 and stack.commits == 1
    assert 2 in L.forwards[-1].tolist()


def test_step_budget_is_global_and_rotates_over_the_layers():
    n_layers = 6
    stack, layers, comp = _stack(n_layers=n_layers, K=2, E=8, spare=2, frequency=1, lag=100,
                                 loads_per_step=1, step_budget=2, commit="ready")
    for st in layers:
        st.layer.imp[:] = [0, 0, 9, 8, 0, 0, 0, 0]    # every layer wants two new experts
    per_step = []
    for _ in range(6):
        before = stack.loads
        stack.step([None] * n_layers, [None] * n_layers)
        per_step.append(stack.loads - before)
    assert max(per_step) <= 2 and sum(per_step) == 2 * n_layers   # two per step until every queue is served
    assert all(len(st.layer.loads) == 2 for st in layers)          # nobody starved
    # without a global budget every layer loads in the same step
    stack2, layers2, _ = _stack(n_layers=n_layers, K=2, E=8, spare=2, frequency=1, lag=100, loads_per_step=1)
    for st in layers2:
        st.layer.imp[:] = [0, 0, 9, 8, 0, 0, 0, 0]
    stack2.step([None] * n_layers, [None] * n_layers)
    assert stack2.loads == n_layers


def test_budget_from_link_rate():
    # 0.8 ms per step at 50 GB/s carries 40 MB, 90 % of it for loads: a little over two 16.8 MB experts
    assert 2.0 <= suggest_step_budget(0.8e-3, 50.0, 16_777_216) < 2.2
    # a 0.2 ms step carries half an expert: the budget is a fraction, i.e. one load every other step
    b = suggest_step_budget(0.2e-3, 50.0, 16_777_216)
    assert 0.5 <= b < 0.6
    stack, layers, _ = _stack(n_layers=2, K=2, E=8, spare=2, frequency=1, lag=100, step_budget=b, commit="ready")
    for st in layers:
        st.layer.imp[:] = [0, 0, 9, 8, 0, 0, 0, 0]
    per_step = []
    for _ in range(8):
        before = stack.loads
        stack.step([None] * 2, [None] * 2)
        per_step.append(stack.loads - before)
    assert max(per_step) == 1 and sum(per_step) == 4 and per_step[0] == 0      # 4 loads wanted, one every other step


def test_layers_may_have_different_budgets():
    """Configuration tuple {frequency, #experts_1..L} (Section 3.3): K is a property of each layer."""
    Ks = [2, 3, 4]
    layers = [LayerState(FakeLayer(K, 8), np.arange(K, dtype=np.int32), np.arange(K, dtype=np.int32),
                         [K], None, None, FakeHost(), FakeHost()) for K in Ks]
    stack = DecodeStack(layers, frequency=1, lag=0, compute_stream=FakeStream(), side_stream=FakeStream(),
                        event_factory=FakeEvent, commit="ready")
    for st in layers:
        st.layer.imp[:] = np.arange(8)[::-1]          # experts 0..K-1 are already the top-K
    stack.step([None] * 3, [None] * 3)
    assert stack.loads == 0
    assert [len(d[3]) for d in stack.decisions] == Ks


def test_asynchronous_decisions_never_wait_for_the_device():
    """async_decide: the scores are only enqueued for copy-out at the decision step; the choice is made at the
    first later step at which the copy's event has fired, with the values of the decision step."""
    made = []

    def factory():
        made.append(FakeEvent())
        return made[-1]

    layers = [LayerState(FakeLayer(2, 6), np.arange(2, dtype=np.int32), np.arange(2, dtype=np.int32), [2],
                         None, None, FakeHost(), FakeHost())]
    stack = DecodeStack(layers, frequency=2, lag=0, compute_stream=FakeStream(), side_stream=FakeStream(),
                        event_factory=factory, commit="ready", async_decide=True,
                        score_alloc=lambda E: torch.zeros((3, E)))
    L = layers[0].layer
    L.imp[:] = [1, 1, 9, 0, 0, 0]
    stack.step([None], [None])                 # step 0: nothing
    stack.step([None], [None])                 # step 1: decision step -> copy enqueued, event pending
    assert len(made) == 1 and not stack.decisions
    stack.step([None], [None])                 # event not fired yet: still no decision, no load
    assert not stack.decisions and stack.loads == 0
    made[0].done = True
    stack.step([None], [None])                 # fired: the decision of step 1 is taken now, the load goes out
    assert [d[0] for d in stack.decisions] == [1] and stack.loads == 1
    assert 2 in stack.decisions[0][3].tolist()
