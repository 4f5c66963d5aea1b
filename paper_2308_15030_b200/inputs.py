"""Seeded synthetic inputs for the Virtual-Expert MoE layer.

This module only draws random numbers and shapes them into the arrays a layer
call needs (tokens, router matrix, expert matrices, expert norms).  It holds none
of the method's arithmetic: no gate, no routing, no FFN.  Both the CPU oracle's
tests and the CUDA path's tests/bench draw their inputs from here so that the two
sides see identical values.

The paper's workloads are Switch-Transformer / GPTSAN checkpoints on text
datasets (Section 4.1).  Neither is available, so the generators below stand in
for them: layer shapes follow those model families, and the routing structure
follows the property the paper relies on (Section 2.2, activation locality:
successive tokens keep asking for the same few experts), realised as a Zipf
popularity law over experts plus runs of tokens that share a preferred expert set.

All floating-point arrays are returned as float32 whose values are exactly
representable in the configuration's storage dtype (fp32 or bf16), so that a
double-precision consumer and a bf16 consumer read the same numbers.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Dict, Optional, Tuple

import numpy as np

F32 = 0
BF16 = 1
ACT_RELU = 0
ACT_SWIGLU = 1


# --------------------------------------------------------------------------- dtype helpers
def round_to_bf16(a: np.ndarray) -> np.ndarray:
    """Round float32 values to the nearest bf16 value (ties to even); result is float32."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    r = (u + np.uint32(0x7FFF) + lsb) & np.uint32(0xFFFF0000)
    return r.view(np.float32)


def bf16_bits(a: np.ndarray) -> np.ndarray:
    """Upper 16 bits of float32 values that are already bf16-representable (uint16)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    u = a.view(np.uint32)
    assert not np.any(u & np.uint32(0xFFFF)), "values are not bf16-representable"
    return (u >> np.uint32(16)).astype(np.uint16)


def bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Inverse of :func:`bf16_bits`: uint16 bf16 patterns -> float32 values."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def store_round(a: np.ndarray, dtype: int) -> np.ndarray:
    a = np.ascontiguousarray(a, dtype=np.float32)
    return round_to_bf16(a) if dtype == BF16 else a


# --------------------------------------------------------------------------- configurations
@dataclass(frozen=True)
class LayerConfig:
    """One MoE-layer workload (shapes, gate flavour and the token recipe)."""
    name: str
    dtype: int
    T: int            # tokens per forward call
    d: int            # d_model
    f: int            # d_ff
    E: int            # experts in the off-the-shelf layer
    k: int            # top-k of the router
    K: int            # resident budget (Virtual-Expert slots)
    act: int = ACT_RELU
    renorm: int = 0   # 1: gate = softmax over the k selected logits
    zipf_s: float = 0.0     # 0 -> no popularity bias
    run_len: int = 32       # tokens that share one preferred expert set
    pref_m: int = 4         # size of the preferred set
    rho: float = 0.9        # probability a token is pulled towards its set
    beta: float = 12.0      # logit boost of the chosen preferred expert
    seed: int = 0
    n_layers: int = 1       # decode configuration: layers per step
    n_steps: int = 1        # decode configuration: steps in the loop

    @property
    def nin(self) -> int:
        return 2 if self.act == ACT_SWIGLU else 1

    @property
    def nmat(self) -> int:
        return self.nin + 1

    @property
    def nb(self) -> int:
        return 2 if self.dtype == BF16 else 4

    def scaled(self, **kw) -> "LayerConfig":
        return replace(self, **kw)


CONFIGS: Dict[str, LayerConfig] = {
    # Single Switch-style layer, fp32.
    "cfg1": LayerConfig("cfg1", F32, T=256, d=768, f=3072, E=8, k=1, K=4, seed=0),
    # Switch-base-64-shaped layer, bf16, Zipf(1.1) popularity with runs of 32 tokens.
    "cfg2": LayerConfig("cfg2", BF16, T=2048, d=768, f=3072, E=64, k=1, K=16,
                        zipf_s=1.1, seed=0),
    # Switch-base-128-shaped prefill, bf16, 16 sequences x 512 tokens, Zipf(1.0).
    "cfg3": LayerConfig("cfg3", BF16, T=8192, d=768, f=3072, E=128, k=1, K=32,
                        zipf_s=1.0, seed=0),
    # Decode loop, bf16: 12 layers, 256 steps, 1..64 tokens per step.
    "cfg4": LayerConfig("cfg4", BF16, T=64, d=1024, f=4096, E=64, k=1, K=16,
                        zipf_s=1.1, seed=0, n_layers=12, n_steps=256),
    # Mixtral-shaped layer, bf16, SwiGLU, top-2 renormalised.
    "cfg5": LayerConfig("cfg5", BF16, T=4096, d=4096, f=14336, E=8, k=2, K=4,
                        act=ACT_SWIGLU, renorm=1, seed=0),
}


# --------------------------------------------------------------------------- layer parameters
def make_router(cfg: LayerConfig, seed: Optional[int] = None) -> np.ndarray:
    """Router matrix Wr [E, d] ~ N(0, 0.1), rounded to the storage dtype."""
    rng = np.random.default_rng([cfg.seed if seed is None else seed, 11])
    return store_round(rng.normal(0.0, 0.1, size=(cfg.E, cfg.d)).astype(np.float32), cfg.dtype)


def make_expert(cfg: LayerConfig, e: int, seed: Optional[int] = None
                ) -> Tuple[np.ndarray, np.ndarray]:
    """Weights of expert ``e``: (w_in [nin, f, d], w_out [d, f]) ~ N(0, 0.02).

    Both matrices are stored with the contraction dimension innermost
    ([out_features, in_features]).  Each expert has its own random stream so a
    caller can materialise only the experts it needs.
    """
    rng = np.random.default_rng([cfg.seed if seed is None else seed, 13, int(e)])
    w_in = rng.standard_normal(size=(cfg.nin, cfg.f, cfg.d), dtype=np.float32)
    w_in *= np.float32(0.02)
    w_out = rng.standard_normal(size=(cfg.d, cfg.f), dtype=np.float32)
    w_out *= np.float32(0.02)
    return store_round(w_in, cfg.dtype), store_round(w_out, cfg.dtype)


def make_enorm(cfg: LayerConfig, seed: Optional[int] = None) -> np.ndarray:
    """Per-expert weight magnitudes ||E_e|| [E] (fp32), supplied to the layer as data.

    Drawn around the Frobenius norm an N(0, 0.02) expert of this shape has,
    0.02*sqrt(nmat*d*f), with a 1 % spread, so that no configuration has to
    materialise all E experts just to know their norms.
    """
    rng = np.random.default_rng([cfg.seed if seed is None else seed, 17])
    base = 0.02 * np.sqrt(float(cfg.nmat) * cfg.d * cfg.f)
    return (base * (1.0 + 0.01 * rng.standard_normal(cfg.E))).astype(np.float32)


def exact_enorm(w_in: np.ndarray, w_out: np.ndarray) -> np.float32:
    """Frobenius norm of all of one expert's parameters (fp64 accumulate -> fp32)."""
    s = np.sum(w_in.astype(np.float64) ** 2) + np.sum(w_out.astype(np.float64) ** 2)
    return np.float32(np.sqrt(s))


# --------------------------------------------------------------------------- tokens
def zipf_law(E: int, s: float) -> np.ndarray:
    p = np.arange(1, E + 1, dtype=np.float64) ** (-float(s))
    return p / p.sum()


def make_tokens(cfg: LayerConfig, Wr: np.ndarray, T: Optional[int] = None,
                seed: Optional[int] = None, return_targets: bool = False):
    """Token matrix x [T, d] ~ N(0,1), optionally biased towards preferred experts.

    With ``cfg.zipf_s > 0`` expert popularity follows Zipf(s) over a random
    ranking of the experts, and every run of ``cfg.run_len`` consecutive tokens
    shares a preferred set of ``cfg.pref_m`` experts drawn from that law.  A token
    is pulled towards one member e of its run's set (probability ``cfg.rho``) by
    adding beta * Wr[e] / ||Wr[e]||^2, which raises its logit for e by exactly
    beta and leaves the others nearly unchanged.  The bias lives in x itself, so
    the layer under test needs no extra input.
    """
    T = cfg.T if T is None else int(T)
    rng = np.random.default_rng([cfg.seed if seed is None else seed, 19])
    x = rng.standard_normal(size=(T, cfg.d), dtype=np.float32)
    target = np.full(T, -1, dtype=np.int32)
    if cfg.zipf_s > 0.0 and T > 0:
        rank_to_id = rng.permutation(cfg.E)
        law = zipf_law(cfg.E, cfg.zipf_s)
        w64 = Wr.astype(np.float64)
        pull = (w64 / np.sum(w64 * w64, axis=1, keepdims=True)).astype(np.float32)
        m = min(cfg.pref_m, cfg.E)
        for r0 in range(0, T, cfg.run_len):
            r1 = min(T, r0 + cfg.run_len)
            pref = rank_to_id[rng.choice(cfg.E, size=m, replace=False, p=law)]
            hit = rng.random(r1 - r0) < cfg.rho
            pick = pref[rng.integers(0, m, size=r1 - r0)]
            for i in range(r1 - r0):
                if hit[i]:
                    target[r0 + i] = pick[i]
                    x[r0 + i] += np.float32(cfg.beta) * pull[pick[i]]
    x = store_round(x, cfg.dtype)
    return (x, target) if return_targets else x


def make_decode_tokens(cfg: LayerConfig, Wr_layers, B: int, n_steps: int,
                       seed: Optional[int] = None) -> np.ndarray:
    """Decode-loop inputs x [n_steps, n_layers, B, d].

    B parallel streams; stream b keeps a preferred expert set per layer that is
    redrawn every ``cfg.run_len`` steps (Zipf popularity as above).  Inputs of
    different layers and steps are independent draws: nothing chains the layers,
    since attention and normalisation are outside the layer under test.
    """
    L = len(Wr_layers)
    rng = np.random.default_rng([cfg.seed if seed is None else seed, 23, B])
    x = rng.standard_normal(size=(n_steps, L, B, cfg.d), dtype=np.float32)
    if cfg.zipf_s > 0.0:
        law = zipf_law(cfg.E, cfg.zipf_s)
        m = min(cfg.pref_m, cfg.E)
        for l in range(L):
            rank_to_id = rng.permutation(cfg.E)
            w64 = Wr_layers[l].astype(np.float64)
            pull = (w64 / np.sum(w64 * w64, axis=1, keepdims=True)).astype(np.float32)
            pref = np.zeros((B, m), dtype=np.int64)
            for s in range(n_steps):
                if s % cfg.run_len == 0:
                    for b in range(B):
                        pref[b] = rank_to_id[rng.choice(cfg.E, size=m, replace=False, p=law)]
                hit = rng.random(B) < cfg.rho
                pick = rng.integers(0, m, size=B)
                for b in range(B):
                    if hit[b]:
                        x[s, l, b] += np.float32(cfg.beta) * pull[pref[b, pick[b]]]
    return store_round(x, cfg.dtype)


# --------------------------------------------------------------------------- weight arenas
def build_arena(cfg: LayerConfig, slot_to_expert, n_phys: Optional[int] = None,
                phys_slot=None, seed: Optional[int] = None
                ) -> Tuple[np.ndarray, np.ndarray]:
    """Pack the listed experts into arenas: in [P, nin, f, d], out [P, d, f] (float32).

    ``phys_slot[s]`` is the arena entry that backs logical slot s (identity by
    default); entries no logical slot points at stay zero.
    """
    K = len(slot_to_expert)
    P = K if n_phys is None else int(n_phys)
    phys = list(range(K)) if phys_slot is None else [int(p) for p in phys_slot]
    a_in = np.zeros((P, cfg.nin, cfg.f, cfg.d), dtype=np.float32)
    a_out = np.zeros((P, cfg.d, cfg.f), dtype=np.float32)
    for s, e in enumerate(slot_to_expert):
        w_in, w_out = make_expert(cfg, int(e), seed)
        a_in[phys[s]] = w_in
        a_out[phys[s]] = w_out
    return a_in, a_out
