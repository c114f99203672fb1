"""Seeded synthetic input generators for the five benchmark workloads.

This module produces INPUTS only: fp32 tensors whose shapes, magnitude
distributions and zero fractions stand in for the activations, weights and
activation gradients the paper logs during training (Section V: tensors of
fully connected and convolution layers).  It contains none of the method's
arithmetic (no rounding, no counting, no contraction) and is the one module
that both the CPU oracle's tests and the CUDA path's tests may import.

Recipe.  "log2|x| ~ N(mu, sigma)" means x = sgn * 2**(mu + sigma*z) with z a
standard normal draw, sgn = +-1 with probability 1/2 (or +1 when
``positive=True``), computed in float64, rounded once to float32, after which
a Bernoulli(p_zero) mask sets exact +0.  All draws come from
``numpy.random.Generator(numpy.random.PCG64(seed))`` in a fixed order, so a
(seed, shape) pair always gives the same bits on every machine.
"""
from __future__ import annotations

from dataclasses import dataclass, field
from typing import Dict, List, Tuple

import numpy as np

# The three 16-bit formats of Table I as (e, m) pairs.
FORMATS: Dict[str, Tuple[int, int]] = {"1/5/10": (5, 10), "1/8/7": (8, 7), "1/6/9": (6, 9)}


def rng_for(seed: int, step: int = 0) -> np.random.Generator:
    """Generator for a workload; ``step`` selects an independent stream per training step."""
    return np.random.Generator(np.random.PCG64([int(seed), int(step)]))


def lognormal_tensor(rng: np.random.Generator, shape, mu: float, sigma: float,
                     p_zero: float = 0.0, positive: bool = False) -> np.ndarray:
    """fp32 tensor with log2|x| ~ N(mu, sigma), random signs, a fraction p_zero of exact zeros."""
    n = int(np.prod(shape))
    out = np.empty(n, dtype=np.float32)
    chunk = 1 << 22  # bounded temporary memory for the 64M-element tensor
    for lo in range(0, n, chunk):
        hi = min(n, lo + chunk)
        z = rng.standard_normal(hi - lo)
        mag = np.exp2(mu + sigma * z)
        if not positive:
            sgn = rng.integers(0, 2, size=hi - lo, dtype=np.int8)
            mag = np.where(sgn == 1, mag, -mag)
        vals = mag.astype(np.float32)
        if p_zero > 0.0:
            mask = rng.random(hi - lo) < p_zero
            vals[mask] = np.float32(0.0)
        out[lo:hi] = vals
    return out.reshape(shape)


def normal_tensor(rng: np.random.Generator, shape, std: float) -> np.ndarray:
    """fp32 tensor with values ~ Normal(0, std) (weights)."""
    return (rng.standard_normal(int(np.prod(shape))) * std).astype(np.float32).reshape(shape)


# ----------------------------------------------------------------------------------------------
# Config 1: small reference case.
# ----------------------------------------------------------------------------------------------
def config1(seed: int = 0):
    """A 256x512 and B 512x256, log2|x| ~ N(-12, 6), 1% exact zeros; format 1/6/9/d, scale 1."""
    rng = rng_for(seed)
    A = lognormal_tensor(rng, (256, 512), -12.0, 6.0, p_zero=0.01)
    B = lognormal_tensor(rng, (512, 256), -12.0, 6.0, p_zero=0.01)
    return {"A": A, "B": B, "fmt": (6, 9), "denormals": 1, "loss_scale": 1.0}


# ----------------------------------------------------------------------------------------------
# Config 2: memory-bound format sweep.
# ----------------------------------------------------------------------------------------------
CONFIG2_N = 64 * 1024 * 1024
CONFIG2_SCALES = (1.0, 2.0 ** 8, 2.0 ** 15)


def config2_tensor(seed: int = 1, n: int = CONFIG2_N) -> np.ndarray:
    """One fp32 tensor, log2|x| ~ N(-18, 8), 0.5% zeros (64 Mi elements by default)."""
    return lognormal_tensor(rng_for(seed), (n,), -18.0, 8.0, p_zero=0.005)


def config2_runs() -> List[Tuple[str, int, int, int, float]]:
    """The 18 (name, e, m, denormals, loss_scale) runs: 3 formats x {d, n} x 3 scales."""
    runs = []
    for name, (e, m) in FORMATS.items():
        for den in (1, 0):
            for s in CONFIG2_SCALES:
                runs.append((f"{name}/{'d' if den else 'n'}@2^{int(np.log2(s))}", e, m, den, s))
    return runs


# ----------------------------------------------------------------------------------------------
# Config 3: BERT-base-shaped fully connected layer.
# ----------------------------------------------------------------------------------------------
def config3(seed: int = 2, tokens: int = 4096, d_in: int = 768, d_out: int = 3072):
    """X tokens x d_in, W d_in x d_out ~ N(0, 0.02), dY tokens x d_out with loss scale 2^10."""
    rng = rng_for(seed)
    X = lognormal_tensor(rng, (tokens, d_in), -3.0, 2.0)
    W = normal_tensor(rng, (d_in, d_out), 0.02)
    dY = lognormal_tensor(rng, (tokens, d_out), -20.0, 4.0)
    return {"X": X, "W": W, "dY": dY, "grad_scale": 2.0 ** 10,
            "variants": [((6, 9), 1), ((6, 9), 0), ((5, 10), 1), ((5, 10), 0)]}


# ----------------------------------------------------------------------------------------------
# Config 4: ResNet-50-shaped convolutions (NCHW).
# ----------------------------------------------------------------------------------------------
@dataclass
class ConvShape:
    n: int
    c_in: int
    h: int
    w: int
    c_out: int
    r: int
    s: int
    pad: int

    @property
    def gemm_mnk(self) -> Tuple[int, int, int]:
        return (self.n * self.h * self.w, self.c_out, self.c_in * self.r * self.s)


CONV3X3 = ConvShape(128, 256, 14, 14, 256, 3, 3, 1)
CONV1X1 = ConvShape(128, 1024, 14, 14, 256, 1, 1, 0)


def config4(shape: ConvShape, seed: int = 3):
    """Post-ReLU activations (half exact zeros, rest 2**N(-2,2) positive), He-normal filters,
    upstream gradients log2|g| ~ N(-20, 4) with loss scale 2^10; format 1/6/9/d."""
    rng = rng_for(seed, step=shape.r)  # independent streams for the 3x3 and the 1x1 layer
    X = lognormal_tensor(rng, (shape.n, shape.c_in, shape.h, shape.w), -2.0, 2.0,
                         p_zero=0.5, positive=True)
    fan_in = shape.c_in * shape.r * shape.s
    Wt = normal_tensor(rng, (shape.c_out, shape.c_in, shape.r, shape.s), float(np.sqrt(2.0 / fan_in)))
    dY = lognormal_tensor(rng, (shape.n, shape.c_out, shape.h, shape.w), -20.0, 4.0)
    return {"X": X, "W": Wt, "dY": dY, "grad_scale": 2.0 ** 10, "fmt": (6, 9), "denormals": 1,
            "shape": shape}


# ----------------------------------------------------------------------------------------------
# Config 5: BERT-large-shaped FC stack, ten steps.
# ----------------------------------------------------------------------------------------------
CONFIG5_LAYERS = (("qkv", 1024, 3072), ("out_proj", 1024, 1024),
                  ("ffn_up", 1024, 4096), ("ffn_down", 4096, 1024))
CONFIG5_TOKENS = 8192
CONFIG5_STEPS = 10


def config5_layer(layer: int, step: int, seed: int = 4, tokens: int = CONFIG5_TOKENS):
    """Fresh tensors of one layer at one step: X N(-3,2), W ~ N(0,0.02), dY N(-24,5), scale 2^16."""
    name, d_in, d_out = CONFIG5_LAYERS[layer]
    rng = rng_for(seed, step=step * len(CONFIG5_LAYERS) + layer)
    X = lognormal_tensor(rng, (tokens, d_in), -3.0, 2.0)
    W = normal_tensor(rng, (d_in, d_out), 0.02)
    dY = lognormal_tensor(rng, (tokens, d_out), -24.0, 5.0)
    return {"name": name, "X": X, "W": W, "dY": dY, "grad_scale": 2.0 ** 16,
            "fmt": (6, 9), "denormals": 1}


# ----------------------------------------------------------------------------------------------
# Structured edge inputs (bit patterns every implementation must get right).
# ----------------------------------------------------------------------------------------------
def edge_bit_patterns() -> np.ndarray:
    """fp32 words covering zeros, fp32 denormals, binade edges, inf and NaN, both signs."""
    pats = [0x00000000, 0x00000001, 0x00000002, 0x007FFFFF, 0x00400000, 0x00800000, 0x00800001,
            0x3F800000, 0x3F7FFFFF, 0x3F800001, 0x7F7FFFFF, 0x7F800000, 0x7F800001, 0x7FC00000,
            0x7FFFFFFF, 0x477FE000, 0x477FF000, 0x477FEFFF, 0x33800000, 0x33000000, 0x33000001,
            0x38800000, 0x387FFFFF, 0x4F7FC000, 0x4F7FE000, 0x2C000000, 0x2B800000, 0x2B800001]
    exps = np.arange(0, 256, dtype=np.uint32) << np.uint32(23)
    fracs = np.array([0, 1, 0x1000, 0x1FFF, 0x2000, 0x2001, 0x3000, 0x3FFF, 0x4000, 0x7FFF, 0x8000,
                      0xFFFF, 0x10000, 0x400000, 0x7FE000, 0x7FF000, 0x7FFFFF], dtype=np.uint32)
    grid = (exps[:, None] | fracs[None, :]).reshape(-1)
    base = np.concatenate([np.array(pats, dtype=np.uint32), grid])
    return np.concatenate([base, base | np.uint32(0x80000000)])
