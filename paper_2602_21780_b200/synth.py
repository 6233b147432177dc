"""Seeded synthetic Q/K/V streams shaped like the paper's workloads.

Input plumbing only: this module holds none of the method's arithmetic.  Both
the CPU oracle's tests and the CUDA path's tests draw their inputs from here so
that they see the same arrays.

Recipe (stands in for real StreamVGGT activations, which need trained weights):
  Q, V ~ N(0,1);
  K = (N(0,1) + mu[h,c]) * m[h,c], with mu ~ N(0, 0.5^2) fixed per
  (layer, head, channel) for the whole stream and m = 10 on 4 seeded channels
  per head, 1 elsewhere -- the channel-wise key outliers of the paper's Fig. 4;
  optional drift: an AR(1) process (rho) on additional per-channel means of
  Q, K and V, stationary standard deviation 0.5.
Values are rounded (nearest-even) to the 16-bit input type once, here; the
float32 arrays returned hold exactly those representable values.

Every (seed, layer, frame, tensor) has its own counter-based Philox stream, so
any frame can be regenerated without generating the ones before it (the drift
means are iterated from frame 0, which costs H*d numbers per frame).
"""
from __future__ import annotations

import numpy as np

BASE_SEED = 20260221
_TENSOR_ID = {"Q": 0, "K": 1, "V": 2, "mu": 3, "outlier": 4, "driftQ": 5, "driftK": 6, "driftV": 7}


def _rng(seed, layer, frame, tensor):
    key = np.array([np.uint64(seed), (np.uint64(layer) << np.uint64(40))
                    | (np.uint64(frame) << np.uint64(8)) | np.uint64(_TENSOR_ID[tensor])],
                   dtype=np.uint64)
    return np.random.Generator(np.random.Philox(key=key))


def round_to_dtype(x, dtype):
    """Round float32 values to fp16 / bf16 (nearest, ties to even) and return
    them as float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "fp16":
        return x.astype(np.float16).astype(np.float32)
    if dtype == "bf16":
        u = x.view(np.uint32).astype(np.uint64)
        u = (u + np.uint64(0x7FFF) + ((u >> np.uint64(16)) & np.uint64(1))) & np.uint64(0xFFFF0000)
        return u.astype(np.uint32).view(np.float32).reshape(x.shape)
    raise ValueError(dtype)


def to_bits16(x, dtype):
    """Bit patterns (uint16) of float32 values already representable in dtype."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    if dtype == "fp16":
        return x.astype(np.float16).view(np.uint16)
    if dtype == "bf16":
        return (x.view(np.uint32) >> np.uint32(16)).astype(np.uint16)
    raise ValueError(dtype)


def from_bits16(u, dtype):
    u = np.ascontiguousarray(u, dtype=np.uint16)
    if dtype == "fp16":
        return u.view(np.float16).astype(np.float32)
    if dtype == "bf16":
        return (u.astype(np.uint32) << np.uint32(16)).view(np.float32)
    raise ValueError(dtype)


class Stream:
    """One layer's stream of per-frame (Q, K, V), each float32 [H, F, d]."""

    def __init__(self, H=16, d=64, F=1374, dtype="bf16", layer=0, seed=BASE_SEED,
                 drift_rho=None, n_outlier=4, outlier_scale=10.0, mu_sigma=0.5):
        self.H, self.d, self.F, self.dtype = H, d, F, dtype
        self.layer, self.seed, self.rho = layer, seed, drift_rho
        r = _rng(seed, layer, 0, "mu")
        self.mu = r.standard_normal((H, 1, d)).astype(np.float32) * np.float32(mu_sigma)
        r = _rng(seed, layer, 0, "outlier")
        self.m = np.ones((H, 1, d), np.float32)
        for h in range(H):
            ch = r.choice(d, size=min(n_outlier, d), replace=False)
            self.m[h, 0, ch] = outlier_scale
        self._drift_cache = {}

    def _drift(self, name, frame):
        """AR(1) per-channel means at `frame` (0-based), iterated from frame 0."""
        if self.rho is None:
            return np.float32(0.0)
        rho = np.float32(self.rho)
        innov = np.float32(np.sqrt(1.0 - float(rho) ** 2) * 0.5)
        last, val = self._drift_cache.get(name, (-1, None))
        if last > frame:
            last, val = -1, None
        for f in range(last + 1, frame + 1):
            eps = _rng(self.seed, self.layer, f, name).standard_normal((self.H, 1, self.d)).astype(np.float32)
            val = eps * np.float32(0.5) if f == 0 else rho * val + innov * eps
        self._drift_cache[name] = (frame, val)
        return val

    def frame(self, t):
        """Frame t (0-based): (Q, K, V) float32 [H, F, d], dtype-representable."""
        shp = (self.H, self.F, self.d)
        q = _rng(self.seed, self.layer, t, "Q").standard_normal(shp, dtype=np.float32)
        k = _rng(self.seed, self.layer, t, "K").standard_normal(shp, dtype=np.float32)
        v = _rng(self.seed, self.layer, t, "V").standard_normal(shp, dtype=np.float32)
        q = q + self._drift("driftQ", t)
        k = (k + self.mu + self._drift("driftK", t)) * self.m
        v = v + self._drift("driftV", t)
        return (round_to_dtype(q, self.dtype), round_to_dtype(k, self.dtype),
                round_to_dtype(v, self.dtype))


# The five workload configurations (shapes, budgets, bit widths).
CONFIGS = {
    0: dict(H=16, d=64, F=261, dtype="fp16", frames=8, L_max=1044, bits=4, layers=1),
    1: dict(H=16, d=64, F=1374, dtype="bf16", frames=64, L_max=21984, bits=4, layers=1),
    2: dict(H=16, d=64, F=1374, dtype="bf16", frames=200, L_max=21984, bits=4, layers=24),
    3: dict(H=16, d=64, F=1374, dtype="bf16", frames=1000, L_max=10992, bits=2, layers=24,
            drift_rho=0.95),
}


def config_stream(cfg_id, layer=0):
    c = CONFIGS[cfg_id]
    return Stream(H=c["H"], d=c["d"], F=c["F"], dtype=c["dtype"], layer=layer,
                  drift_rho=c.get("drift_rho"))
