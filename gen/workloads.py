"""Seeded synthetic workloads for the CriticalKV compression step.

This module only draws random tensors and rounds them to the storage type.
It contains none of the method's arithmetic (no softmax, no projection, no
selection): both the CPU oracle and the CUDA library consume the arrays it
returns, byte for byte, and neither of them is imported here.

Shapes follow the models the paper evaluates (Llama-3.1-8B / Mistral-7B:
32 query heads, 8 KV heads, head_dim 128, d_model 4096; Qwen2.5-32B: 40 query
heads, 8 KV heads, d_model 5120; observation window 32 and max-pool kernel 7,
Section 4.1).  Datasets and trained weights are replaced by distributions
with the structure that matters to the path:

* keys ~ N(0,1) with 4 outlier channels per KV head scaled by 8 (the massive
  key channels real models have);
* window queries = 0.5 * (mean of 8 random context keys of the head's KV head)
  + N(0, 1/32) noise per row, then rescaled so that the logits of one row over
  random keys have a prescribed standard deviation ``s``.  Gaussian logits give
  log-normal (heavy-tailed) attention weights whose top-5% share is
  Phi(s - 1.645), so ``s`` sets the attention concentration without the
  generator ever computing an attention weight;
* values ~ N(0,1) with a per-token log-normal row scale (so value-row norms
  spread over orders of magnitude);
* W_O ~ N(0, 1/d_model) with a per-head scale drawn from U[0.5, 2].

Layouts (row-major, innermost contiguous):
  Qw [Hq, w, dh]   K, V [Hkv, n, dh]   WO [Hq, dh, dm]
where WO[h] is rows h*dh .. (h+1)*dh of the (Hq*dh) x dm output projection.
"""
from __future__ import annotations

import math
from dataclasses import dataclass, field, replace
from statistics import NormalDist

import numpy as np

OUTLIER_CHANNELS = 4
OUTLIER_SCALE = 8.0
ANCHOR_KEYS = 8
ANCHOR_WEIGHT = 0.5
QUERY_NOISE_STD = 0.5 / math.sqrt(8.0)
Z95 = 1.6448536269514722  # 95th percentile of the standard normal


@dataclass(frozen=True)
class Workload:
    """One named configuration (per layer shapes and selection parameters)."""

    name: str
    cfg_id: int
    dtype: str            # "f32" or "bf16": storage type of Qw, K, V, WO
    Hq: int
    Hkv: int
    dh: int
    dm: int
    n: int
    w: int
    kp: int
    budget_mode: str      # "uniform" | "adaptive"
    budget: int           # uniform: B per KV head; adaptive: B_total per layer
    alpha: float = 0.5
    eps: float = 1e-4
    layers: int = 1
    value_sigma: float = 1.0
    top5_share: tuple = (0.7, 0.7)   # per-layer target drawn uniformly in this range
    extra: dict = field(default_factory=dict)

    @property
    def G(self) -> int:
        return self.Hq // self.Hkv

    @property
    def scale(self) -> float:
        return 1.0 / math.sqrt(self.dh)

    @property
    def btot(self) -> int:
        """Retained entries per layer (sum over KV heads)."""
        return self.budget * self.Hkv if self.budget_mode == "uniform" else self.budget

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


def _cfgs():
    c = {}
    c[0] = Workload("cfg0_tiny_f32", 0, "f32", 4, 2, 64, 256, 512, 16, 5, "uniform", 128)
    c[1] = Workload("cfg1_llama8b_4k", 1, "bf16", 32, 8, 128, 4096, 4096, 32, 7, "uniform",
                    int(0.2 * 4096))
    c[2] = Workload("cfg2_mistral7b_32k", 2, "bf16", 32, 8, 128, 4096, 32768, 32, 7, "uniform",
                    int(0.4 * 32768))
    c[3] = Workload("cfg3_llama8b_32k_32layers_adaptive", 3, "bf16", 32, 8, 128, 4096, 32768, 32, 7,
                    "adaptive", int(0.2 * 8 * 32768), layers=32, top5_share=(0.4, 0.9))
    c[4] = Workload("cfg4_qwen32b_128k_64layers", 4, "bf16", 40, 8, 128, 5120, 131072, 64, 7,
                    "uniform", int(0.1 * 131072), layers=64, value_sigma=1.5)
    return c


CONFIGS = _cfgs()


def config(cfg_id: int) -> Workload:
    return CONFIGS[cfg_id]


# ----------------------------------------------------------------------------
# storage rounding
# ----------------------------------------------------------------------------
def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bfloat16 (nearest even); returns the 16-bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    rounded = u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))
    return (rounded >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    """Exact widening of bfloat16 bit patterns to float32."""
    return (b.astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed: int, stream: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([int(seed), int(stream)])))


def concentration_to_logit_std(share: float) -> float:
    """Logit standard deviation whose log-normal weights put ``share`` of the
    mass on the top 5% of keys: share = Phi(s - z95)."""
    return Z95 + NormalDist().inv_cdf(share)


@dataclass
class LayerInputs:
    """Inputs of one layer.  ``*_store`` are the arrays handed to the CUDA
    library (float32, or uint16 bfloat16 bit patterns); ``Qw, K, V, WO`` are
    the same values widened exactly to float32 for the CPU oracle."""

    wl: Workload
    layer: int
    seed: int
    Qw: np.ndarray
    K: np.ndarray
    V: np.ndarray
    WO: np.ndarray
    Qw_store: np.ndarray
    K_store: np.ndarray
    V_store: np.ndarray
    WO_store: np.ndarray
    logit_std: float
    share_target: float


def _store(x: np.ndarray, dtype: str):
    if dtype == "f32":
        x = np.ascontiguousarray(x, dtype=np.float32)
        return x, x
    bits = f32_to_bf16_bits(x)
    return bf16_bits_to_f32(bits), bits


def make_layer(wl: Workload, layer: int = 0, *, want=("Qw", "K", "V", "WO")) -> LayerInputs:
    """Draw the four input tensors of one layer (seed = 10000*cfg + layer)."""
    seed = 10000 * wl.cfg_id + layer
    Hq, Hkv, G, dh, dm, n, w = wl.Hq, wl.Hkv, wl.G, wl.dh, wl.dm, wl.n, wl.w

    r_meta = _rng(seed, 0)
    lo, hi = wl.top5_share
    share = float(lo + (hi - lo) * r_meta.random())
    s_target = concentration_to_logit_std(share)

    # keys: N(0,1), 4 outlier channels per KV head scaled by 8
    r_k = _rng(seed, 1)
    K = r_k.standard_normal((Hkv, n, dh), dtype=np.float32)
    chan_std = np.ones((Hkv, dh), dtype=np.float32)
    for g in range(Hkv):
        ch = r_meta.choice(dh, size=OUTLIER_CHANNELS, replace=False)
        K[g][:, ch] *= np.float32(OUTLIER_SCALE)
        chan_std[g, ch] = OUTLIER_SCALE

    # window queries: anchor mean + noise, rescaled to the target logit std
    r_q = _rng(seed, 2)
    Qw = np.empty((Hq, w, dh), dtype=np.float32)
    n_ctx = max(n - w, 1)
    for h in range(Hq):
        g = h // G
        anchors = r_q.integers(0, n_ctx, size=ANCHOR_KEYS)
        m = K[g][anchors].mean(axis=0)
        q = ANCHOR_WEIGHT * m[None, :] + QUERY_NOISE_STD * r_q.standard_normal((w, dh), dtype=np.float32)
        row_std = np.sqrt(((q * chan_std[g][None, :]) ** 2).sum(axis=1))  # std of q.k over random keys
        gamma = s_target / (wl.scale * row_std)
        Qw[h] = q * gamma[:, None].astype(np.float32)

    # values: N(0,1) with a per-token log-normal row scale
    r_v = _rng(seed, 3)
    V = r_v.standard_normal((Hkv, n, dh), dtype=np.float32)
    row_scale = np.exp(wl.value_sigma * r_v.standard_normal((Hkv, n, 1), dtype=np.float32))
    V *= row_scale

    # output projection: N(0, 1/dm), per-head scale U[0.5, 2]
    r_o = _rng(seed, 4)
    if "WO" in want:
        WO = r_o.standard_normal((Hq, dh, dm), dtype=np.float32)
        u = r_o.uniform(0.5, 2.0, size=(Hq, 1, 1)).astype(np.float32)
        WO *= u / np.float32(math.sqrt(dm))
    else:
        WO = np.zeros((Hq, dh, 1), dtype=np.float32)

    Qw_f, Qw_s = _store(Qw, wl.dtype)
    K_f, K_s = _store(K, wl.dtype)
    V_f, V_s = _store(V, wl.dtype)
    WO_f, WO_s = _store(WO, wl.dtype)
    return LayerInputs(wl, layer, seed, Qw_f, K_f, V_f, WO_f, Qw_s, K_s, V_s, WO_s, s_target, share)


def small_workload(*, dtype="f32", Hq=4, Hkv=2, dh=64, dm=128, n=300, w=8, kp=5,
                   budget_mode="uniform", budget=40, alpha=0.5, cfg_id=90, **kw) -> Workload:
    """Ad-hoc small workload for tests (ragged sizes, edge cases)."""
    return Workload(f"small_{cfg_id}", cfg_id, dtype, Hq, Hkv, dh, dm, n, w, kp, budget_mode, budget,
                    alpha=alpha, **kw)
