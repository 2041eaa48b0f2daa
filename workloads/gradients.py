"""Seeded gradient streams (inputs only; no optimizer arithmetic).

Every stream is a pure function of (seed, layer index, call index): it uses
numpy's counter-based Philox generator keyed on those integers, so the oracle
and the CUDA path can each ask for "the gradient of layer l at call c" and get
identical bits.  Values are produced in float64, rounded once to float32 and,
for bf16 streams, rounded to bfloat16 with round-to-nearest-even; the float32
array that is returned holds exactly the rounded values.
"""
from __future__ import annotations

import numpy as np

from .configs import Workload

_TAG_NOISE, _TAG_FACTOR_A, _TAG_FACTOR_B, _TAG_WEIGHT = 1, 2, 3, 4


def _rng(seed: int, layer: int, call: int, tag: int) -> np.random.Generator:
    key = (int(seed) & 0xFFFFFFFFFFFFFFFF, ((int(layer) + 1) << 8) | tag)
    return np.random.Generator(np.random.Philox(key=np.array(key, dtype=np.uint64),
                                                counter=np.array([0, 0, 0, int(call)], dtype=np.uint64)))


def to_bf16_bits(x32: np.ndarray) -> np.ndarray:
    """float32 -> bfloat16 bit patterns (uint16), round-to-nearest-even."""
    u = np.ascontiguousarray(x32, dtype=np.float32).view(np.uint32)
    rounding = ((u >> 16) & 1) + np.uint32(0x7FFF)
    return ((u + rounding) >> 16).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (bits.astype(np.uint32) << 16).view(np.float32)


def initial_weight(w: Workload, layer: int) -> np.ndarray:
    """W_0 ~ N(0, 0.02^2), float32."""
    l = w.layers[layer]
    return (0.02 * _rng(w.seed + 1, layer, 0, _TAG_WEIGHT).standard_normal((l.m, l.n))).astype(np.float32)


class GradientStream:
    """g_c for one layer of a workload; `call` counts from 1."""

    def __init__(self, w: Workload, layer: int):
        self.w, self.layer = w, layer
        spec = w.layers[layer]
        self.m, self.n = spec.m, spec.n
        self._A = self._B = None
        if w.grad_kind == "lowrank_noise":
            # Signal factors drawn once per layer: a persistent signal subspace.
            self._A = _rng(w.seed, layer, 0, _TAG_FACTOR_A).standard_normal((self.m, w.grad_rank))
            self._B = _rng(w.seed, layer, 0, _TAG_FACTOR_B).standard_normal((self.n, w.grad_rank))
        if w.grad_kind == "integer_subspace":
            # Gradients confined to fixed rank-r row and column spaces, with entries that are small integers
            # times grad_scale (a power of two): exactly representable in bf16, so that products and short
            # sums of them are exact in fp32 and the factors G G^T, G^T G have exactly rank r on both sides.
            self._A = _rng(w.seed, layer, 0, _TAG_FACTOR_A).integers(-1, 2, (self.m, w.grad_rank)).astype(np.float64)
            self._B = _rng(w.seed, layer, 0, _TAG_FACTOR_B).integers(-1, 2, (self.n, w.grad_rank)).astype(np.float64)

    def f64(self, call: int) -> np.ndarray:
        w = self.w
        r = _rng(w.seed, self.layer, call, _TAG_NOISE)
        if w.grad_kind == "iid_normal":
            return w.grad_scale * r.standard_normal((self.m, self.n))
        if w.grad_kind == "lowrank_noise":
            return self._A @ self._B.T + w.grad_scale * r.standard_normal((self.m, self.n))
        if w.grad_kind == "integer_subspace":
            C = r.integers(-1, 2, (w.grad_rank, w.grad_rank)).astype(np.float64)
            return w.grad_scale * (self._A @ C @ self._B.T)
        if w.grad_kind == "student_t":
            return w.grad_scale * r.standard_t(3.0, size=(self.m, self.n))
        raise ValueError(w.grad_kind)

    def __call__(self, call: int) -> np.ndarray:
        """float32 array holding the values exactly as the optimizer receives them."""
        g = self.f64(call).astype(np.float32)
        if self.w.grad_dtype == "bf16":
            g = bf16_bits_to_f32(to_bf16_bits(g))
        return g

    def bits(self, call: int) -> np.ndarray:
        """The buffer handed to the library: float32, or uint16 bf16 patterns."""
        g = self.f64(call).astype(np.float32)
        return to_bf16_bits(g) if self.w.grad_dtype == "bf16" else g
