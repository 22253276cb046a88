"""Seeded synthetic inputs for the INT8 SSD layer.

This module serves both the CUDA path and the CPU oracle and therefore holds
none of the method's arithmetic: it only names the workload shapes and draws
floating-point tensors with the value structure the paper reports for Mamba-2
activations (a few outlier channels in X, unit-scale B and C, small positive
time steps after softplus, negative per-head decay rates).

Symbols follow the paper (Section 4.1): batch B, length L, heads H, head
dimension P, state dimension N, groups G, chunk length l (called Q here),
c = L / Q chunks, D = H * P channels.
"""
from __future__ import annotations

from dataclasses import dataclass

import numpy as np


@dataclass(frozen=True)
class SSDConfig:
    name: str
    batch: int
    seqlen: int
    nheads: int
    headdim: int
    dstate: int
    ngroups: int
    chunk: int
    outlier_frac: float
    outlier_gain: float
    seed: int
    decode_steps: int = 0  # > 0: recurrent-mode workload, seqlen is 1 token per step

    @property
    def nchunks(self) -> int:
        return self.seqlen // self.chunk

    @property
    def channels(self) -> int:
        return self.nheads * self.headdim

    @property
    def tokens(self) -> int:
        return self.batch * self.seqlen

    def replace(self, **kw) -> "SSDConfig":
        d = dict(self.__dict__)
        d.update(kw)
        return SSDConfig(**d)


# The five seeded workloads (shapes of Mamba-2 130M / 2.7B / 8B SSD layers).
CONFIGS = {
    "cfg0": SSDConfig("cfg0", 1, 512, 4, 64, 64, 1, 64, 0.02, 20.0, 0),
    "cfg1": SSDConfig("cfg1", 1, 2048, 24, 64, 128, 1, 256, 0.02, 20.0, 1),
    "cfg2": SSDConfig("cfg2", 8, 2048, 80, 64, 128, 1, 256, 0.01, 50.0, 2),
    "cfg3": SSDConfig("cfg3", 4, 8192, 128, 64, 128, 8, 256, 0.01, 50.0, 3),
    "cfg4": SSDConfig("cfg4", 64, 1, 80, 64, 128, 1, 256, 0.01, 50.0, 4, decode_steps=256),
}

# tensor ids: one independent random stream per tensor
_TID = {"x": 0, "B": 1, "C": 2, "dt": 3, "A": 4, "D": 5, "outliers": 6, "init": 7}


def _rng(seed: int, tid: int, step: int = 0) -> np.random.Generator:
    return np.random.default_rng([int(seed), int(tid), int(step)])


def outlier_channels(cfg: SSDConfig) -> np.ndarray:
    """Indices of the channels (of D = H*P) that carry the outlier gain."""
    d = cfg.channels
    k = max(1, int(np.ceil(cfg.outlier_frac * d)))
    return np.sort(_rng(cfg.seed, _TID["outliers"]).permutation(d)[:k])


def _softplus(v: np.ndarray) -> np.ndarray:
    return np.logaddexp(0.0, v)


def make_prefill(cfg: SSDConfig) -> dict:
    """fp32 tensors of one SSD layer forward: x [B,L,H,P], B/C [B,L,G,N],
    dt [B,L,H] (already positive), A [H] (< 0), D [H]."""
    b, L, H, P, N, G = cfg.batch, cfg.seqlen, cfg.nheads, cfg.headdim, cfg.dstate, cfg.ngroups
    x = _rng(cfg.seed, _TID["x"]).standard_normal((b, L, H * P), dtype=np.float32)
    x[:, :, outlier_channels(cfg)] *= np.float32(cfg.outlier_gain)
    x = x.reshape(b, L, H, P)
    Bm = _rng(cfg.seed, _TID["B"]).standard_normal((b, L, G, N), dtype=np.float32)
    Cm = _rng(cfg.seed, _TID["C"]).standard_normal((b, L, G, N), dtype=np.float32)
    dt = _softplus(_rng(cfg.seed, _TID["dt"]).standard_normal((b, L, H)) - 3.0).astype(np.float32)
    A = (-np.exp(_rng(cfg.seed, _TID["A"]).uniform(0.0, np.log(16.0), H))).astype(np.float32)
    D = _rng(cfg.seed, _TID["D"]).standard_normal(H).astype(np.float32)
    return {"x": x, "B": Bm, "C": Cm, "dt": dt, "A": A, "D": D}


def make_decode_step(cfg: SSDConfig, step: int) -> dict:
    """fp32 tensors of one recurrent-mode token: x [B,H,P], B/C [B,G,N], dt [B,H]."""
    b, H, P, N, G = cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate, cfg.ngroups
    x = _rng(cfg.seed, _TID["x"], step + 1).standard_normal((b, H * P), dtype=np.float32)
    x[:, outlier_channels(cfg)] *= np.float32(cfg.outlier_gain)
    x = x.reshape(b, H, P)
    Bm = _rng(cfg.seed, _TID["B"], step + 1).standard_normal((b, G, N), dtype=np.float32)
    Cm = _rng(cfg.seed, _TID["C"], step + 1).standard_normal((b, G, N), dtype=np.float32)
    dt = _softplus(_rng(cfg.seed, _TID["dt"], step + 1).standard_normal((b, H)) - 3.0).astype(np.float32)
    return {"x": x, "B": Bm, "C": Cm, "dt": dt}


def make_decode_params(cfg: SSDConfig) -> dict:
    """Per-head parameters shared by every decode step: A [H] (< 0), D [H]."""
    H = cfg.nheads
    A = (-np.exp(_rng(cfg.seed, _TID["A"]).uniform(0.0, np.log(16.0), H))).astype(np.float32)
    D = _rng(cfg.seed, _TID["D"]).standard_normal(H).astype(np.float32)
    return {"A": A, "D": D}


def make_init_state(cfg: SSDConfig, scale: float = 1.0) -> np.ndarray:
    """A non-zero initial state [B,H,P,N] for the hand-off cases."""
    s = _rng(cfg.seed, _TID["init"]).standard_normal(
        (cfg.batch, cfg.nheads, cfg.headdim, cfg.dstate), dtype=np.float32)
    return (s * np.float32(scale)).astype(np.float32)
