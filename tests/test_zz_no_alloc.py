"""The routing entry point that allocates nothing (collected last on purpose).

Some callers may not call cudaMalloc: a plug-in inside an application that owns all
device memory, a real-time loop that must stay off the driver's allocation lock.  For
them the library offers swapmoe_route_static, whose scratch is a fixed array inside the
library image.  This test calls it through the C ABI twice in a row - a large batch and
then a smaller one, so the second call meets the first call's leftovers in the shared
scratch - and checks every output against the regular entry point (swapmoe_forward and
its taps) on the same inputs.  fp32 layers run the same router kernel on both sides, so
everything must agree to the last bit; bf16 layers route through the tensor-core router
on the regular path, so logits and gates agree to the tolerances of the parity tests
and indices are compared wherever the deciding logit margin is not a near-tie.
Each call's outputs are also held against the CPU oracle (fed the call's own logits):
indices, counts and offsets bit for bit, gate values, token norms and Eq. (1) within
the tolerances of the parity tests.
"""
import numpy as np
import pytest

from paper_2308_15030_b200 import inputs as I

pytestmark = pytest.mark.gpu


def _route_static(case, T):
    import torch
    from paper_2308_15030_b200 import binding
    cfg = case.cfg
    dev = "cuda"
    e2s = np.full(cfg.E, -1, np.int32)
    e2s[case.s2e] = np.arange(cfg.K, dtype=np.int32)
    t = {
        "logits": torch.full((T, cfg.E), float("nan"), device=dev),
        "uidx": torch.full((T, cfg.k), -7, dtype=torch.int32, device=dev),
        "ugate": torch.full((T, cfg.k), float("nan"), device=dev),
        "midx": torch.full((T, cfg.k), -7, dtype=torch.int32, device=dev),
        "mgate": torch.full((T, cfg.k), float("nan"), device=dev),
        "slot": torch.full((T, cfg.k), -7, dtype=torch.int32, device=dev),
        "xnorm": torch.full((T,), float("nan"), device=dev),
        "count": torch.full((cfg.K,), -7, dtype=torch.int32, device=dev),
        "offset": torch.full((cfg.K + 1,), -7, dtype=torch.int32, device=dev),
        "imp": torch.zeros(cfg.E, device=dev),
    }
    binding.route_static(case.d_x[:T], case.d_Wr, torch.from_numpy(e2s).cuda(),
                         torch.from_numpy(case.enorm).cuda(), cfg.k, cfg.K, cfg.dtype, cfg.renorm,
                         t["logits"], t["uidx"], t["ugate"], t["midx"], t["mgate"], t["slot"],
                         t["xnorm"], t["count"], t["offset"], t["imp"])
    torch.cuda.synchronize()
    return {k: v.cpu().numpy() for k, v in t.items()}


def _compare_with_oracle(case, T, got):
    """The arithmetic itself: logits against the fp64 product, then routing from those very logits."""
    import oracle
    from harness import TOL_GATE_ABS, TOL_IMP_REL, TOL_LOGIT_REL
    cfg = case.cfg
    x = case.x[:T]
    ref_l = oracle.logits(x, case.Wr)
    assert np.max(np.abs(got["logits"] - ref_l)) <= TOL_LOGIT_REL * np.max(np.abs(ref_l))
    uidx, ugate = oracle.gate(got["logits"], cfg.k, cfg.renorm)
    res = np.zeros(cfg.E, np.int32); res[case.s2e] = 1
    midx, mgate = oracle.gate(got["logits"], cfg.k, cfg.renorm, allowed=res)
    slot = oracle.invert_slot_table(case.s2e, cfg.E)[midx]
    count, offset, _, _ = oracle.permute(slot, cfg.K)
    for name, ref in (("uidx", uidx), ("midx", midx), ("slot", slot), ("count", count), ("offset", offset)):
        assert np.array_equal(got[name], ref.reshape(got[name].shape)), name
    assert np.max(np.abs(got["ugate"] - ugate)) <= TOL_GATE_ABS
    assert np.max(np.abs(got["mgate"] - mgate)) <= TOL_GATE_ABS
    xn = np.linalg.norm(x.astype(np.float64), axis=1)
    assert np.max(np.abs(got["xnorm"] - xn)) <= 1e-5 * max(1.0, xn.max())
    imp = oracle.importance(x, uidx, ugate, case.enorm)
    assert np.max(np.abs(got["imp"] - imp)) <= TOL_IMP_REL * imp.max()


def _compare(case, T, got, exact):
    _compare_with_oracle(case, T, got)
    L = case.layer
    L.read_importance(reset=True)
    L.forward(case.d_x, case.d_out, n_tokens=T)
    ref = {n: L.tap(n) for n in ("logits", "uidx", "ugate", "midx", "mgate", "slot", "xnorm", "count", "offset")}
    ref["imp"] = L.read_importance(reset=True)
    if exact:
        for n, r in ref.items():
            assert np.array_equal(got[n], r), n
        return
    scale = np.max(np.abs(ref["logits"]))
    assert np.max(np.abs(got["logits"] - ref["logits"])) <= 1e-5 * scale
    # tokens whose deciding margins are clear on the regular path's logits
    srt = np.sort(ref["logits"], axis=1)[:, ::-1]
    res = np.zeros(case.cfg.E, bool); res[case.s2e] = True
    srt_m = np.sort(np.where(res[None, :], ref["logits"], -np.inf), axis=1)[:, ::-1]
    k = case.cfg.k
    clear = (np.min(srt[:, :k] - srt[:, 1:k + 1], axis=1) > 1e-4 * scale) & \
            (np.min(srt_m[:, :k] - srt_m[:, 1:k + 1], axis=1) > 1e-4 * scale)
    assert clear.mean() > 0.9
    for n in ("uidx", "midx", "slot"):
        assert np.array_equal(got[n][clear], ref[n][clear]), n
    # logits may differ by 1e-5 * scale between the two routers, which moves a softmax value by
    # at most about that much in absolute terms
    for n in ("ugate", "mgate"):
        assert np.max(np.abs(got[n][clear] - ref[n][clear])) <= 1e-6 + 2e-5 * scale, n
    assert np.max(np.abs(got["xnorm"] - ref["xnorm"])) <= 1e-5 * ref["xnorm"].max()
    if clear.all():
        assert np.array_equal(got["count"], ref["count"]) and np.array_equal(got["offset"], ref["offset"])
    assert got["count"].sum() == T * k and got["offset"][-1] == T * k
    assert np.max(np.abs(got["imp"] - ref["imp"])) <= 1e-3 * ref["imp"].max()


@pytest.mark.parametrize("dtype,k,renorm", [(I.F32, 1, 0), (I.F32, 2, 1), (I.BF16, 1, 0)])
def test_route_static_matches_forward_twice_in_a_row(monkeypatch, dtype, k, renorm):
    from harness import Case
    cfg = I.LayerConfig("noalloc", dtype, T=1000, d=256, f=256, E=48, k=k, K=9, renorm=renorm,
                        zipf_s=1.1, seed=4)
    # fp32: with the small-batch routers off, `forward` runs the very kernel `route_static` runs, so
    # the two must agree bit for bit; bf16 layers are compared within the routers' tolerance
    if dtype == I.F32:
        monkeypatch.setenv("SWAPMOE_SMALL_ROUTER", "0")
    case = Case(cfg)
    exact = dtype == I.F32
    first = _route_static(case, 1000)          # 32 router blocks leave their partials in the scratch
    second = _route_static(case, 333)          # fewer blocks: must not be confused by the leftovers
    _compare(case, 1000, first, exact)
    _compare(case, 333, second, exact)


def test_route_static_rejects_sizes_beyond_its_scratch():
    import torch
    from paper_2308_15030_b200 import binding
    T = binding.ROUTE_STATIC_MAX_TOKENS + 1
    x = torch.zeros((T, 64), device="cuda")
    Wr = torch.zeros((4, 64), device="cuda")
    z = torch.zeros(4 * T, device="cuda")
    zi = torch.zeros(4 * T, dtype=torch.int32, device="cuda")
    with pytest.raises(binding.SwapMoEError) as e:
        binding.route_static(x, Wr, zi, z, 1, 2, binding.F32, 0, z, zi, z, zi, z, zi, z, zi, zi, z)
    assert e.value.status == -3
