"""Shared set-up of the GPU parity tests: seeded inputs -> CUDA layer and -> CPU oracle."""
from __future__ import annotations

import numpy as np

import oracle
from paper_2308_15030_b200 import binding, inputs as I

TOL_OUT = {I.F32: 1e-4, I.BF16: 2e-2}      # max|err| / ||ref||_inf  (spec tolerances)
TOL_LOGIT_REL = 1e-5                        # relative to ||logits||_inf
TOL_GATE_ABS = 1e-6
TOL_IMP_REL = 1e-4                          # relative to max importance


def to_device(a: np.ndarray, dtype: int):
    import torch
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == I.BF16:
        return torch.from_numpy(I.bf16_bits(a).view(np.int16)).view(torch.bfloat16).cuda()
    return torch.from_numpy(a).cuda()


def to_host_f32(t) -> np.ndarray:
    import torch
    if t.dtype == torch.bfloat16:
        return I.bits_to_f32(t.view(torch.int16).cpu().numpy().view(np.uint16))
    return t.float().cpu().numpy()


def choose_resident(cfg, x, Wr, enorm):
    """Top-K experts by the oracle's importance (Eq. 1) of this batch."""
    lg = oracle.logits(x, Wr)
    uidx, ugate = oracle.gate(lg, cfg.k, cfg.renorm)
    return oracle.topk_importance(oracle.importance(x, uidx, ugate, enorm), cfg.K)


class Case:
    """Inputs of one layer call, materialised on the host and on the GPU."""

    def __init__(self, cfg, T=None, s2e=None, phys=None, spare=0, max_tokens=None):
        import torch
        self.cfg = cfg
        self.T = cfg.T if T is None else T
        self.Wr = I.make_router(cfg)
        self.enorm = I.make_enorm(cfg)
        self.x = I.make_tokens(cfg, self.Wr, self.T)
        if s2e is None:
            s2e = choose_resident(cfg, self.x, self.Wr, self.enorm) if self.T > 0 \
                else np.arange(cfg.K, dtype=np.int32)
        self.s2e = np.asarray(s2e, np.int32)
        self.P = cfg.K + spare
        self.phys = np.arange(cfg.K, dtype=np.int32) if phys is None else np.asarray(phys, np.int32)
        self.a_in, self.a_out = I.build_arena(cfg, self.s2e, self.P, self.phys)
        self.d_Wr = to_device(self.Wr, cfg.dtype)
        self.d_x = to_device(self.x, cfg.dtype) if self.T > 0 else \
            torch.zeros((0, cfg.d), dtype=torch.bfloat16 if cfg.dtype == I.BF16 else torch.float32,
                        device="cuda")
        self.d_in = to_device(self.a_in, cfg.dtype)
        self.d_out_w = to_device(self.a_out, cfg.dtype)
        self.d_out = torch.full((max(self.T, 1), cfg.d), float("nan"), dtype=self.d_x.dtype, device="cuda")
        self.layer = binding.Layer(cfg.E, cfg.d, cfg.f, cfg.k, cfg.K, cfg.dtype, cfg.act, cfg.renorm,
                                   max_tokens=max(self.T, 1) if max_tokens is None else max_tokens,
                                   spare_slots=spare)
        self.layer.set_router(self.d_Wr, self.enorm)
        self.layer.set_resident(self.s2e, self.d_in, self.d_out_w, self.phys)

    def run(self, ext_logits=None):
        import torch
        if ext_logits is None:
            self.layer.forward(self.d_x, self.d_out, n_tokens=self.T)
        else:
            self.d_ext = torch.from_numpy(np.ascontiguousarray(ext_logits, np.float32)).cuda()
            self.layer.forward_from_logits(self.d_x, self.d_ext, self.d_out)
        torch.cuda.synchronize()
        return to_host_f32(self.d_out[: self.T])

    def oracle(self, gpu_logits, token_subset=None, imp=None):
        return oracle.forward(self.x, self.Wr, self.enorm, self.s2e, self.a_in, self.a_out,
                              k=self.cfg.k, act=self.cfg.act, renorm=self.cfg.renorm,
                              phys_slot=self.phys, ext_logits=gpu_logits, token_subset=token_subset,
                              imp=imp)


def check_against_oracle(case: Case, out_gpu: np.ndarray, token_subset=None, check_logits=True,
                         imp_before=None):
    """Two-stage comparison: logits vs the oracle's double product, then everything
    else against the oracle run FROM THE GPU'S fp32 logits (so routing is compared
    on identical logits and a routing flip cannot pass as a value error)."""
    cfg, L = case.cfg, case.layer
    assert L.device_status() == (0, 0), "a bounded device wait gave up"
    logits = L.tap("logits")
    if check_logits:
        ref_l = oracle.logits(case.x, case.Wr)
        err = np.max(np.abs(logits.astype(np.float64) - ref_l))
        assert err <= TOL_LOGIT_REL * np.max(np.abs(ref_l)), ("logits", err)
    r = case.oracle(logits, token_subset=token_subset, imp=imp_before)
    for name in ("uidx", "midx", "slot", "count", "offset", "perm", "inv"):
        got = L.tap(name)
        assert np.array_equal(got, r[name].reshape(got.shape)), name
    for name in ("ugate", "mgate"):
        assert np.max(np.abs(L.tap(name).astype(np.float64) - r[name])) <= TOL_GATE_ABS, name
    xn = np.linalg.norm(case.x.astype(np.float64), axis=1)
    assert np.max(np.abs(L.tap("xnorm") - xn)) <= 1e-5 * max(1.0, xn.max())
    rows = np.arange(case.T) if token_subset is None else np.asarray(token_subset)
    ref = r["out"][rows]
    scale = np.max(np.abs(ref))
    err = np.max(np.abs(out_gpu[rows].astype(np.float64) - ref))
    assert np.all(np.isfinite(out_gpu[rows]))
    assert err <= TOL_OUT[cfg.dtype] * scale, ("out", err / scale)
    imp = L.read_importance()
    assert np.max(np.abs(imp.astype(np.float64) - r["imp"])) <= TOL_IMP_REL * max(1e-30, r["imp"].max()), "imp"
    return {"out_rel_err": float(err / scale), "oracle": r}
