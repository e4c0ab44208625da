"""Seeded synthetic inputs for the LTE layer.

This module holds none of the method's arithmetic: it only draws tensors with the
value distributions of the benchmark configurations and rounds them to the storage
dtype.  Both the CUDA path's tests and the CPU oracle consume the identical bits.

Recipe: every tensor of batch element ``b`` comes from its own NumPy PCG64 stream
``default_rng([seed, tag, b])`` (``tag`` names the tensor), ``standard_normal`` in
float32, scaled, then rounded to nearest-even bf16 when the configuration is bf16.
Per-batch streams make any subset of sequences reproducible without drawing the
rest.  q, k ~ N(0,1)/d^0.25 (N(0,1) for the tiny fp32 case), v ~ N(0,1),
conv weights ~ N(0, sigma_w) in fp32 (never rounded), upstream dO ~ N(0,1).
"""
from dataclasses import dataclass, replace

import numpy as np

_TAG = {"q": 0, "k": 1, "v": 2, "w": 3, "dO": 4, "bias": 5}


@dataclass(frozen=True)
class Config:
    name: str
    dtype: str          # "f32" or "bf16"
    B: int
    H: int
    d: int
    T: int
    W: int
    R: int
    K: int              # taps of the single-layer scorer
    sigma_w: float
    qk_unit: bool = False   # True: q,k ~ N(0,1); False: N(0,1)/d^0.25
    sink: int = 0
    steps: int = 0      # decode steps after the T-token prompt

    def with_(self, **kw):
        return replace(self, **kw)


CONFIGS = {
    "C1": Config("C1", "f32", 1, 2, 32, 128, 16, 8, 5, 0.1, qk_unit=True),
    "C2": Config("C2", "bf16", 4, 16, 64, 4096, 128, 128, 7, 0.05),
    "C3": Config("C3", "bf16", 1, 16, 128, 32768, 512, 512, 7, 0.05),
    "C4": Config("C4", "bf16", 128, 16, 64, 8192, 128, 128, 7, 0.05, steps=256),
    "C5": Config("C5", "bf16", 8, 16, 64, 2048, 64, 64, 7, 0.05),
}


def round_bf16(x):
    """Round float32 values to the nearest bf16 (ties to even); result stays float32."""
    x = np.ascontiguousarray(x, dtype=np.float32)
    u = x.view(np.uint32).astype(np.uint64)
    u = (u + 0x7FFF + ((u >> 16) & 1)) & 0xFFFF0000
    return u.astype(np.uint32).view(np.float32).reshape(x.shape)


def _normal(seed, tag, b, shape):
    return np.random.default_rng([seed, _TAG[tag], b]).standard_normal(shape, dtype=np.float32)


def tensor(cfg, tag, seed=0, batch=None, T=None):
    """[len(batch), H, T, d] float32 array for tag in {"q","k","v","dO"} (bf16-rounded if cfg is bf16)."""
    T = cfg.T if T is None else T
    batch = range(cfg.B) if batch is None else batch
    out = np.stack([_normal(seed, tag, b, (cfg.H, T, cfg.d)) for b in batch])
    if tag in ("q", "k") and not cfg.qk_unit:
        out *= np.float32(cfg.d ** -0.25)
    return round_bf16(out) if cfg.dtype == "bf16" else out


def conv_weights(cfg, seed=0):
    """Scorer weights [H, K, 2d] float32 ~ N(0, sigma_w)."""
    return (_normal(seed, "w", 0, (cfg.H, cfg.K, 2 * cfg.d)) * np.float32(cfg.sigma_w)).astype(np.float32)


def make(cfg, seed=0, batch=None, T=None, with_dO=False):
    """dict(q, k, v, w[, dO]) for ``cfg``; ``T`` overrides the length (e.g. prompt + decode steps)."""
    out = {t: tensor(cfg, t, seed, batch, T) for t in ("q", "k", "v")}
    out["w"] = conv_weights(cfg, seed)
    if with_dO:
        out["dO"] = tensor(cfg, "dO", seed, batch, T)
    return out


def query_sample(cfg, nq, seed=0, batch=None):
    """[len(batch), H, nq] int32: nq distinct query positions per head, ascending."""
    batch = range(cfg.B) if batch is None else batch
    out = np.empty((len(batch), cfg.H, nq), np.int32)
    for a, b in enumerate(batch):
        rng = np.random.default_rng([seed, 99, b])
        for h in range(cfg.H):
            out[a, h] = np.sort(rng.choice(cfg.T, size=nq, replace=False)).astype(np.int32)
    return out
