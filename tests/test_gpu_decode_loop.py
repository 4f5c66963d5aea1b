"""Decode loop with asynchronous expert swapping (needs a B200).

The CUDA stack records which slot table every (step, layer) forward used; the oracle
replays that trace for output parity, and the importance windows / top-K decisions are
checked against the oracle's own Eq. (1) accumulation.
"""
import numpy as np
import pytest

import oracle
from paper_2308_15030_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _build(cfg, L, B, steps, frequency, lag, spare, loads_per_step=1, Ks=None, **stack_kw):
    """Ks: per-layer resident budgets (default cfg.K everywhere); stack_kw goes to DecodeStack."""
    import torch
    from harness import to_device
    from paper_2308_15030_b200 import binding
    from paper_2308_15030_b200.decode import DecodeStack, LayerState
    host = []
    states = []
    tdt = torch.bfloat16 if cfg.dtype == I.BF16 else torch.float32
    Ks = [cfg.K] * L if Ks is None else list(Ks)
    for l in range(L):
        c = cfg.scaled(seed=1000 + l)
        K = Ks[l]
        Wr, enorm = I.make_router(c), I.make_enorm(c)
        w_in = np.empty((cfg.E, cfg.nin, cfg.f, cfg.d), np.float32)
        w_out = np.empty((cfg.E, cfg.d, cfg.f), np.float32)
        for e in range(cfg.E):
            w_in[e], w_out[e] = I.make_expert(c, e)
        if cfg.dtype == I.BF16:
            h_in = torch.from_numpy(I.bf16_bits(w_in).view(np.int16)).view(torch.bfloat16).pin_memory()
            h_out = torch.from_numpy(I.bf16_bits(w_out).view(np.int16)).view(torch.bfloat16).pin_memory()
        else:
            h_in, h_out = torch.from_numpy(w_in).pin_memory(), torch.from_numpy(w_out).pin_memory()
        P = K + spare
        a_in = torch.zeros((P, cfg.nin, cfg.f, cfg.d), dtype=tdt, device="cuda")
        a_out = torch.zeros((P, cfg.d, cfg.f), dtype=tdt, device="cuda")
        s2e = np.arange(K, dtype=np.int32)                      # arbitrary initial resident set
        a_in[:K].copy_(h_in[:K]); a_out[:K].copy_(h_out[:K])
        layer = binding.Layer(cfg.E, cfg.d, cfg.f, cfg.k, K, cfg.dtype, cfg.act, cfg.renorm,
                              max_tokens=B, spare_slots=spare)
        d_Wr = to_device(Wr, cfg.dtype)
        layer.set_router(d_Wr, enorm)
        states.append(LayerState(layer, s2e, np.arange(K, dtype=np.int32), list(range(K, P)),
                                 a_in, a_out, h_in, h_out, enorm=enorm))
        host.append(dict(Wr=Wr, enorm=enorm, w_in=w_in, w_out=w_out, d_Wr=d_Wr))
    x = I.make_decode_tokens(cfg, [h["Wr"] for h in host], B, steps)      # [steps, L, B, d]
    d_x = to_device(x.reshape(-1, cfg.d), cfg.dtype).reshape(steps, L, B, cfg.d)
    torch.cuda.synchronize()
    stack = DecodeStack(states, frequency=frequency, loads_per_step=loads_per_step, lag=lag, **stack_kw)
    return stack, host, x, d_x


def _check_replay(cfg, stack, host, x, outs):
    from harness import TOL_OUT
    for entry in stack.trace:
        s, l, s2e, phys = entry
        assert len(set(phys.tolist())) == len(phys) and len(set(s2e.tolist())) == len(s2e)
        ref = _replay(cfg, host, x, entry)["out"]
        err = np.max(np.abs(outs[s, l] - ref)) / max(1e-30, np.max(np.abs(ref)))
        assert err <= TOL_OUT[cfg.dtype], (s, l, err)


def _run(stack, d_x, cfg, steps, L, B):
    import torch
    outs = torch.empty((steps, L, B, cfg.d), dtype=d_x.dtype, device="cuda")
    for s in range(steps):
        stack.step([d_x[s, l] for l in range(L)], [outs[s, l] for l in range(L)])
    torch.cuda.synchronize()
    return outs


def _replay(cfg, host, x, entry, token_subset=None):
    s, l, s2e, _ = entry
    h = host[l]
    return oracle.forward(x[s, l], h["Wr"], h["enorm"], s2e, h["w_in"][s2e], h["w_out"][s2e],
                          k=cfg.k, act=cfg.act, renorm=cfg.renorm, token_subset=token_subset)


def test_decode_loop_small_full_replay():
    from harness import to_host_f32, TOL_OUT
    cfg = I.LayerConfig("dec", I.BF16, T=5, d=128, f=256, E=16, k=1, K=4, zipf_s=1.1, seed=0)
    L, B, steps, freq, lag = 3, 5, 40, 8, 2
    stack, host, x, d_x = _build(cfg, L, B, steps, freq, lag, spare=2)
    outs = to_host_f32(_run(stack, d_x, cfg, steps, L, B).reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
    assert len(stack.trace) == steps * L
    assert stack.loads > 0                                   # experts were swapped in
    assert any(not np.array_equal(t[2], np.arange(cfg.K)) for t in stack.trace)
    assert all(st.layer.device_status() == (0, 0) for st in stack.layers)
    # 1. every forward used exactly the table the trace says, with the right weights behind it
    win = [np.zeros(cfg.E) for _ in range(L)]
    dec = {(n, l): (imp, top) for n, l, imp, top in stack.decisions}
    for entry in stack.trace:
        s, l, s2e, phys = entry
        assert len(set(phys.tolist())) == cfg.K and len(set(s2e.tolist())) == cfg.K
        r = _replay(cfg, host, x, entry)
        ref = r["out"]
        err = np.max(np.abs(outs[s, l] - ref)) / max(1e-30, np.max(np.abs(ref)))
        assert err <= TOL_OUT[cfg.dtype], (s, l, err)
        win[l] += r["imp"]
        # 2. importance window and top-K decision
        if (s, l) in dec:
            imp_gpu, top_gpu = dec[(s, l)]
            assert np.max(np.abs(imp_gpu - win[l])) <= 1e-4 * win[l].max()
            srt = np.sort(win[l])[::-1]
            if srt[cfg.K - 1] - srt[cfg.K] > 1e-4 * srt[0]:
                assert set(top_gpu.tolist()) == set(oracle.topk_importance(win[l], cfg.K).tolist())
            win[l][:] = 0
    # 3. the loop converges onto the important experts: late tables differ from the initial one
    last = [t for t in stack.trace if t[0] == steps - 1]
    assert any(set(t[2].tolist()) != set(range(cfg.K)) for t in last)


def test_decode_loop_never_serves_a_half_loaded_expert():
    """Aggressive schedule (decision every 2 steps, commit lag 0, one spare): outputs must still
    match the replay of the recorded tables at every step."""
    from harness import to_host_f32, TOL_OUT
    cfg = I.LayerConfig("dec2", I.BF16, T=9, d=128, f=256, E=12, k=2, K=3, renorm=1, act=I.ACT_SWIGLU,
                        zipf_s=1.2, run_len=4, seed=5)
    L, B, steps = 2, 9, 24
    stack, host, x, d_x = _build(cfg, L, B, steps, frequency=2, lag=0, spare=1, loads_per_step=2)
    outs = to_host_f32(_run(stack, d_x, cfg, steps, L, B).reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
    assert stack.loads >= 2
    for entry in stack.trace:
        s, l, _, _ = entry
        ref = _replay(cfg, host, x, entry)["out"]
        err = np.max(np.abs(outs[s, l] - ref)) / max(1e-30, np.max(np.abs(ref)))
        assert err <= TOL_OUT[cfg.dtype], (s, l, err)


def test_cfg4_shape_sampled():
    """Full cfg4 layer shape (d 1024, d_ff 4096, E 64, K 16), two layers, B = 64 and B = 1;
    routing compared on every step, FFN values on sampled (step, layer, token) triples."""
    from harness import to_host_f32, TOL_OUT
    base = I.CONFIGS["cfg4"]
    rng = np.random.default_rng(3)
    for B, steps in ((64, 20), (1, 20)):
        cfg = base.scaled(T=B)
        L = 2
        stack, host, x, d_x = _build(cfg, L, B, steps, frequency=8, lag=2, spare=2)
        outs = to_host_f32(_run(stack, d_x, cfg, steps, L, B).reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
        assert stack.loads > 0 and stack.bytes_loaded == stack.loads * 2 * 1024 * 4096 * 2
        picks = rng.choice(len(stack.trace), size=6, replace=False)
        for i in picks:
            entry = stack.trace[i]
            s, l, _, _ = entry
            sub = np.sort(rng.choice(B, size=min(B, 4), replace=False)).astype(np.int32)
            ref = _replay(cfg, host, x, entry, token_subset=sub)["out"][sub]
            err = np.max(np.abs(outs[s, l][sub] - ref)) / max(1e-30, np.max(np.abs(ref)))
            assert err <= TOL_OUT[cfg.dtype], (B, s, l, err)
        del stack, host


def test_decode_loop_through_cuda_graph_matches_replay():
    """The step's forwards captured as a CUDA graph (fixed buffers), table flips outside it."""
    import torch
    from harness import to_host_f32, TOL_OUT
    cfg = I.LayerConfig("decg", I.BF16, T=6, d=128, f=256, E=16, k=1, K=4, zipf_s=1.1, seed=2)
    L, B, steps = 2, 6, 24
    stack, host, x, d_x = _build(cfg, L, B, steps, frequency=4, lag=1, spare=2)
    xbuf = torch.empty((L, B, cfg.d), dtype=d_x.dtype, device="cuda")
    obuf = torch.empty_like(xbuf)
    stack.graph_buffers = (xbuf, obuf)
    outs = torch.empty((steps, L, B, cfg.d), dtype=d_x.dtype, device="cuda")
    for s in range(steps):
        stack.step_graph(d_x[s], record=True)
        outs[s].copy_(obuf)
    torch.cuda.synchronize()
    outs = to_host_f32(outs.reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
    assert stack.loads > 0
    for entry in stack.trace:
        s, l, _, _ = entry
        ref = _replay(cfg, host, x, entry)["out"]
        err = np.max(np.abs(outs[s, l] - ref)) / max(1e-30, np.max(np.abs(ref)))
        assert err <= TOL_OUT[cfg.dtype], (s, l, err)


def test_commit_when_ready_with_a_global_load_budget():
    """Fig. 5 (ii), amortised + asynchronous: at most two loads per step over all layers, and a slot flips
    only once its copy has landed (nothing ever waits for a copy); the recorded tables replay exactly."""
    from harness import to_host_f32
    cfg = I.LayerConfig("decr", I.BF16, T=6, d=128, f=256, E=16, k=1, K=4, zipf_s=1.1, seed=7)
    L, B, steps = 4, 6, 48
    stack, host, x, d_x = _build(cfg, L, B, steps, frequency=4, lag=1, spare=2, step_budget=2, commit="ready")
    outs = to_host_f32(_run(stack, d_x, cfg, steps, L, B).reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
    assert stack.loads > 0 and stack.commits > 0 and stack.stalls == 0
    assert stack.commits + sum(len(st.pending) for st in stack.layers) == stack.loads
    _check_replay(cfg, stack, host, x, outs)
    assert any(set(t[2].tolist()) != set(range(cfg.K)) for t in stack.trace if t[0] == steps - 1)


def test_static_pruning_policy():
    """Section 4.1 "Pruning": the K experts with the largest ||E_i|| are installed once and never change."""
    import oracle
    from harness import to_host_f32
    cfg = I.LayerConfig("decp", I.BF16, T=5, d=128, f=256, E=16, k=1, K=4, zipf_s=1.1, seed=8)
    L, B, steps = 2, 5, 10
    stack, host, x, d_x = _build(cfg, L, B, steps, frequency=2, lag=0, spare=1, policy="static_pruning")
    loads0 = stack.loads
    outs = to_host_f32(_run(stack, d_x, cfg, steps, L, B).reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
    assert stack.loads == loads0 and not stack.decisions          # no updates during the loop
    for s, l, s2e, _ in stack.trace:
        assert set(s2e.tolist()) == set(oracle.topk_importance(host[l]["enorm"], cfg.K).tolist())
    _check_replay(cfg, stack, host, x, outs)


def test_on_demand_policy():
    """Section 2.1 / 4.1 "On demand": an expert the off-the-shelf gate asks for is loaded before the layer
    runs (blocking), so with no more distinct requests than slots the output is the unrestricted layer's."""
    import oracle
    from harness import to_host_f32, TOL_OUT
    cfg = I.LayerConfig("deco", I.BF16, T=3, d=128, f=256, E=16, k=1, K=4, zipf_s=1.1, seed=9)
    L, B, steps = 2, 3, 16
    stack, host, x, d_x = _build(cfg, L, B, steps, frequency=1 << 30, lag=0, spare=1, policy="on_demand")
    outs = to_host_f32(_run(stack, d_x, cfg, steps, L, B).reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
    assert stack.blocking_loads > 0 and stack.misses >= stack.blocking_loads and stack.requests == steps * L * B
    _check_replay(cfg, stack, host, x, outs)
    for s, l, s2e, _ in stack.trace:
        h = host[l]
        uidx, _ = oracle.gate(oracle.logits(x[s, l], h["Wr"]), cfg.k, cfg.renorm)
        assert set(uidx.reshape(-1).tolist()) <= set(s2e.tolist())          # B <= K: every request is served
        full = oracle.forward(x[s, l], h["Wr"], h["enorm"], np.arange(cfg.E), h["w_in"], h["w_out"],
                              k=cfg.k, act=cfg.act, renorm=cfg.renorm)      # all experts resident
        # the gate value differs (softmax over the resident set, not over all experts); the expert does not
        r = _replay(cfg, host, x, (s, l, s2e, None))
        assert np.array_equal(r["midx"], full["midx"])


def test_heterogeneous_budgets_in_one_graph():
    """Section 3.3: the configuration is {frequency, #experts_1..L}.  Layers with K = 8, 12, 16, 24 slots run as
    ONE CUDA graph per step; tables flip outside the graph; every (step, layer) output replays."""
    import torch
    from harness import to_host_f32
    cfg = I.LayerConfig("dech", I.BF16, T=16, d=128, f=256, E=32, k=1, K=8, zipf_s=1.1, seed=10)
    Ks = [8, 12, 16, 24] * 3
    L, B, steps = len(Ks), 16, 12
    stack, host, x, d_x = _build(cfg, L, B, steps, frequency=4, lag=1, spare=2, Ks=Ks, step_budget=3,
                                 commit="ready")
    xbuf = torch.empty((L, B, cfg.d), dtype=d_x.dtype, device="cuda")
    obuf = torch.empty_like(xbuf)
    stack.graph_buffers = (xbuf, obuf)
    outs = torch.empty((steps, L, B, cfg.d), dtype=d_x.dtype, device="cuda")
    for s in range(steps):
        stack.step_graph(d_x[s], record=True)
        outs[s].copy_(obuf)
    torch.cuda.synchronize()
    outs = to_host_f32(outs.reshape(-1, cfg.d)).reshape(steps, L, B, cfg.d)
    assert stack.loads > 0
    assert [len(t[2]) for t in stack.trace[:L]] == Ks
    _check_replay(cfg, stack, host, x, outs)
