"""Seeded synthetic workloads shaped like the paper's Wan2.1-1.3B video-DiT layers.

This module only draws inputs.  It contains none of the method's arithmetic (no token
rule, no feature map, no attention) so that the CPU oracle and the CUDA library can
both be fed from it without sharing any code of the method.

Recipe (stand-in for the paper's Wan2.1 / VBench workloads, which need weights and
prompts that are not available offline): a 480x832 video is VAE-compressed 8x spatially
and 4x temporally and patchified 1x2x2, giving 30x52 tokens per latent frame and
(frames - 1) / 4 + 1 latent frames.  Q and K are N(0,1) draws whose (token, head)
vectors are scaled to unit RMS (the effect of the DiT's QK-norm: scores q.k/sqrt(d) are
roughly N(0,1)); V is N(0,1); the feature-map weights are Glorot-uniform per head.
Every tensor is rounded to bf16 (round-to-nearest-even) on the host; the float64 view
handed to the oracle holds exactly those bf16 values.
"""
from __future__ import annotations

import dataclasses
import functools
import math

import numpy as np


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    B: int
    H: int
    d: int
    F: int
    grid: tuple          # (T, Hg, Wg) latent grid, w fastest
    block: tuple         # (bt, bh, bw) spatial block
    rate: int            # R: 1 = full softmax, 0 = pure linear, else softmax rate 1/R
    seed: int
    rms_norm_qk: bool = True
    degree: int = 2      # polynomial degree P of the feature map
    layers: int = 1      # depth of the feature map's embedding network
    hidden: int = 0      # hidden width of a two-layer network (0: equal to F)
    bias: bool = False   # embedding layers carry a bias

    @property
    def hidden_width(self) -> int:
        return self.hidden if self.hidden > 0 else self.F

    @property
    def N(self) -> int:
        return self.grid[0] * self.grid[1] * self.grid[2]

    def with_rate(self, rate: int, seed: int | None = None) -> "Workload":
        return dataclasses.replace(self, rate=rate, seed=self.seed if seed is None else seed,
                                   name=f"{self.name}/R{rate}")


# The five benchmark configurations.  Seeds are 1000 * config number (+ layer for the stack).
CONFIGS = {
    "tiny": Workload("tiny", B=1, H=2, d=64, F=64, grid=(4, 16, 16), block=(2, 4, 4),
                     rate=32, seed=0, rms_norm_qk=False),
    "wan17": Workload("wan17", B=1, H=12, d=128, F=128, grid=(5, 30, 52), block=(1, 6, 8),
                      rate=8, seed=2000),
    "wan81": Workload("wan81", B=1, H=12, d=128, F=128, grid=(21, 30, 52), block=(1, 6, 8),
                      rate=8, seed=3000),
    "wan161cfg": Workload("wan161cfg", B=2, H=12, d=128, F=128, grid=(41, 30, 52),
                          block=(1, 6, 8), rate=16, seed=5000),
}

# The headline layer with wider feature maps ("Characterization of phi"; table of phi sizes): the paper's default
# map, two layers d -> 2d -> 2d with polynomial degree 2, and a one-layer map of the same output width.
VARIANTS = {
    "wan81_paper_phi": Workload("wan81_paper_phi", B=1, H=12, d=128, F=256, grid=(21, 30, 52), block=(1, 6, 8),
                                rate=8, seed=3100, layers=2, hidden=256),
    "wan81_f256": Workload("wan81_f256", B=1, H=12, d=128, F=256, grid=(21, 30, 52), block=(1, 6, 8),
                           rate=8, seed=3200),
}

STACK_RATES = (1, 4, 8, 16, 0)   # rate index -> R for the 30-layer block-rate stack
STACK_LAYERS = 30


def splitmix64_stream(seed: int):
    """Generator of the SplitMix64 sequence (a public counter-based PRNG)."""
    mask = (1 << 64) - 1
    state = seed & mask
    while True:
        state = (state + 0x9E3779B97F4A7C15) & mask
        zz = state
        zz = ((zz ^ (zz >> 30)) * 0xBF58476D1CE4E5B9) & mask
        zz = ((zz ^ (zz >> 27)) * 0x94D049BB133111EB) & mask
        yield zz ^ (zz >> 31)


def stack_schedule(seed: int = 0, layers: int = STACK_LAYERS):
    """Per-layer hybrid rates of the cost-aware block-rate stack (seeded schedule)."""
    gen = splitmix64_stream(seed)
    return [STACK_RATES[next(gen) % len(STACK_RATES)] for _ in range(layers)]


def stack_errors(seed: int = 0, layers: int = STACK_LAYERS) -> np.ndarray:
    """Synthetic per-block errors e_ir [layers][len(STACK_RATES)] for the block-rate selection: zero at
    rate 1, growing towards sparser rates, with a per-block sensitivity spread over a decade (stand-ins
    for the distillation errors, which need the trained model)."""
    rng = np.random.default_rng(9000 + seed)
    steps = rng.uniform(0.2, 1.0, (layers, len(STACK_RATES)))
    steps[:, 0] = 0.0
    return np.cumsum(steps, axis=1) * np.exp(rng.uniform(np.log(0.3), np.log(3.0), (layers, 1)))


def stack_layer(layer: int, seed: int = 0) -> Workload:
    """Workload of one layer of the 30-layer stack (headline shape, scheduled rate)."""
    rate = stack_schedule(seed)[layer]
    base = CONFIGS["wan81"]
    return dataclasses.replace(base, name=f"stack/L{layer}/R{rate}", rate=rate,
                               seed=4000 + layer)


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even); returns the uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    bias = ((u >> np.uint32(16)) & np.uint32(1)) + np.uint32(0x7FFF)
    return ((u + bias) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(b: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(b, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f32(b).astype(np.float64)


@functools.lru_cache(maxsize=2)
def _draw(wl: Workload):
    """The raw draws of one workload: q, k, v as bf16 bit patterns, the weights still in float32
    (the gain on W_q is applied before rounding).  Kept for the last two workloads: the tests ask
    for the same layer several times (other gains, fewer heads)."""
    rng = np.random.Generator(np.random.PCG64(wl.seed))
    shape = (wl.B, wl.H, wl.N, wl.d)
    out = {}
    for name in ("q", "k", "v"):
        x = rng.standard_normal(shape, dtype=np.float32)
        if wl.rms_norm_qk and name in ("q", "k"):
            x /= np.sqrt(np.mean(np.square(x, dtype=np.float32), axis=-1, keepdims=True))
        out[name] = f32_to_bf16_bits(x)
        del x
    hid = wl.hidden_width
    first_out = hid if wl.layers == 2 else wl.F
    a = math.sqrt(6.0 / (wl.d + first_out))
    out["wq"] = rng.uniform(-a, a, size=(wl.H, first_out, wl.d)).astype(np.float32)
    out["wk"] = rng.uniform(-a, a, size=(wl.H, first_out, wl.d)).astype(np.float32)
    if wl.layers == 2:
        # second layer [H, F, hidden], drawn after the first layers (which then map d -> hidden)
        a2 = math.sqrt(6.0 / (hid + wl.F))
        out["wq2"] = rng.uniform(-a2, a2, size=(wl.H, wl.F, hid)).astype(np.float32)
        out["wk2"] = rng.uniform(-a2, a2, size=(wl.H, wl.F, hid)).astype(np.float32)
    if wl.bias:
        # small biases of either sign, drawn last: bq1, bk1 (, bq2, bk2)
        out["bq1"] = rng.uniform(-0.1, 0.1, size=(wl.H, first_out)).astype(np.float32)
        out["bk1"] = rng.uniform(-0.1, 0.1, size=(wl.H, first_out)).astype(np.float32)
        if wl.layers == 2:
            out["bq2"] = rng.uniform(-0.1, 0.1, size=(wl.H, wl.F)).astype(np.float32)
            out["bk2"] = rng.uniform(-0.1, 0.1, size=(wl.H, wl.F)).astype(np.float32)
    return out


def teacher_output(wl: Workload) -> np.ndarray:
    """Stand-in for the teacher block's attention output y of the distillation step ("Attention Distillation"; the
    real one needs the pretrained model): N(0, 1/4) draws [B, H, N, d] from a stream of its own (seed wl.seed + 77),
    rounded to bf16; returns the bit patterns."""
    rng = np.random.Generator(np.random.PCG64(wl.seed + 77))
    return f32_to_bf16_bits(0.5 * rng.standard_normal((wl.B, wl.H, wl.N, wl.d), dtype=np.float32))


WEIGHT_NAMES = ("wq", "wk", "wq2", "wk2", "bq1", "bk1", "bq2", "bk2")


def generate(wl: Workload, wq_gain: float = 1.0, heads: int | None = None):
    """Draw one layer's inputs.  Returns a dict of uint16 arrays holding bf16 bit patterns:

      q, k, v : [B, H, N, d]
      wq, wk  : [H, F, d]                     (wl.layers == 2: [H, hidden, d], and wq2, wk2 : [H, F, hidden])
      bq1, bk1 (, bq2, bk2) : [H, width]      (only when wl.bias)

    Draw order is Q, K, V, W_q, W_k (, W_q2, W_k2) (, biases) from numpy's PCG64 seeded with `wl.seed`.
    `wq_gain` multiplies the LAST layer of the query map (weights and bias) before rounding (used by the
    tests to make the softmax and the linear branch carry comparable weight; ReLU is positively
    homogeneous, so this scales the activation a by the gain).  `heads` (optional) keeps only the
    first few heads, after drawing all of them, so that a reduced case sees the same values.
    """
    raw = _draw(wl)
    g = np.float32(wq_gain)
    last_w, last_b = ("wq2", "bq2") if wl.layers == 2 else ("wq", "bq1")
    out = {}
    for name, x in raw.items():
        if name in ("q", "k", "v"):
            out[name] = x.copy()          # the cached draw itself is never handed out
        else:
            out[name] = f32_to_bf16_bits(x * g if name in (last_w, last_b) else x)
    if heads is not None and heads < wl.H:
        for name in ("q", "k", "v"):
            out[name] = np.ascontiguousarray(out[name][:, :heads])
        for name in WEIGHT_NAMES:
            if name in out:
                out[name] = np.ascontiguousarray(out[name][:heads])
    return out
