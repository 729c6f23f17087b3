"""Seeded synthetic inputs for the expert-parallel dispatch/combine path.

This module only draws random routing tables, weights and activations; it holds
none of the method's arithmetic (no counting, no slots, no reduction), so both the
CPU oracle's tests and the CUDA path's tests may import it.

Recipe (numpy ``Generator(PCG64)`` seeded with ``SeedSequence([seed, config id,
array id])``; seed 0 unless overridden):

* ``x``            [T, H] fp32 N(0,1) narrowed to bf16 by torch (round to nearest even)
* ``topk_weights`` [T, K] softmax over K iid N(0,1) logits, fp32
* ``topk_idx``     [T, K] int32, K distinct experts per token, in sample order
    - ``uniform``: first K entries of the argsort of E iid uniforms
    - ``zipf``   : Plackett-Luce sample (Gumbel top-K) with p_e proportional to
                   (pi(e)+1)^-1.1, pi a seeded permutation of the experts
                   (``zipf_identity`` keeps pi = identity: the stress case in which
                   the lowest ranks hold the hot experts)
    - ``burst``  : uniform, then a seeded subset of exactly round(0.1*T) tokens gets
                   expert 0 as its k=0 pick unless the token already picked it
* ``out``          [rows, H] bf16 N(0,1): synthetic expert outputs for combine

The shapes follow the MoE families the paper names in Section 2.1 (8 experts
top-2; 8 of 256; 10 of 512); they stand in for the paper's model workloads.
"""
from __future__ import annotations

from dataclasses import dataclass, replace

import numpy as np
import torch

_ARRAY_IDS = {"x": 0, "topk_idx": 1, "topk_weights": 2, "out": 3, "burst": 4, "perm": 5}


@dataclass(frozen=True)
class EPConfig:
    name: str
    T: int          # tokens (all source ranks together)
    H: int          # hidden size, bf16 elements per row
    E: int          # experts
    K: int          # experts picked per token
    R: int          # logical expert-parallel ranks
    routing: str    # uniform | zipf | zipf_identity | burst
    config_id: int
    host_staged: bool = False

    @property
    def shape(self):
        return (self.T, self.K, self.H, self.E, self.R)


CONFIGS = {
    "C1": EPConfig("C1", T=64, H=256, E=8, K=2, R=2, routing="uniform", config_id=1),
    "C2": EPConfig("C2", T=256, H=4096, E=8, K=2, R=8, routing="uniform", config_id=2),
    "C3": EPConfig("C3", T=4096, H=2048, E=128, K=8, R=8, routing="zipf", config_id=3),
    "C4": EPConfig("C4", T=8192, H=7168, E=256, K=8, R=8, routing="burst", config_id=4),
    "C5": EPConfig("C5", T=4096, H=2048, E=128, K=8, R=8, routing="zipf", config_id=3,
                   host_staged=True),
}


def custom_config(T, H, E, K, R, routing="uniform", config_id=99, name="custom"):
    return EPConfig(name, T=T, H=H, E=E, K=K, R=R, routing=routing, config_id=config_id)


def _rng(seed: int, config_id: int, array: str) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([seed, config_id, _ARRAY_IDS[array]]))


def to_bf16_bits(a_f32: np.ndarray) -> np.ndarray:
    """fp32 array -> bf16 bit patterns (uint16), narrowed by torch's CPU cast."""
    t = torch.from_numpy(np.ascontiguousarray(a_f32, dtype=np.float32)).to(torch.bfloat16)
    return t.view(torch.int16).numpy().view(np.uint16)


def bf16_bits_to_f32(bits_u16: np.ndarray) -> np.ndarray:
    """bf16 bit patterns (uint16) -> fp32 values, widened by torch's CPU cast."""
    t = torch.from_numpy(np.ascontiguousarray(bits_u16).view(np.int16)).view(torch.bfloat16)
    return t.to(torch.float32).numpy()


def expert_popularity(cfg: EPConfig, seed: int = 0) -> np.ndarray:
    """Probability of each expert under the config's routing recipe (first pick)."""
    if cfg.routing in ("uniform", "burst"):
        return np.full(cfg.E, 1.0 / cfg.E)
    if cfg.routing == "zipf":
        pi = _rng(seed, cfg.config_id, "perm").permutation(cfg.E)
    elif cfg.routing == "zipf_identity":
        pi = np.arange(cfg.E)
    else:
        raise ValueError(f"unknown routing {cfg.routing!r}")
    p = (pi + 1.0) ** -1.1
    return p / p.sum()


def make_topk_idx(cfg: EPConfig, seed: int = 0) -> np.ndarray:
    T, K, E = cfg.T, cfg.K, cfg.E
    if K > E:
        raise ValueError("K distinct experts per token need K <= E")
    rng = _rng(seed, cfg.config_id, "topk_idx")
    if cfg.routing in ("uniform", "burst"):
        keys = rng.random((T, E))
        idx = np.argsort(keys, axis=1, kind="stable")[:, :K]
    elif cfg.routing in ("zipf", "zipf_identity"):
        logp = np.log(expert_popularity(cfg, seed))
        g = rng.gumbel(size=(T, E))
        idx = np.argsort(-(logp[None, :] + g), axis=1, kind="stable")[:, :K]
    else:
        raise ValueError(f"unknown routing {cfg.routing!r}")
    idx = np.ascontiguousarray(idx, dtype=np.int32)
    if cfg.routing == "burst" and T > 0:
        n_hot = int(round(0.1 * T))
        hot = _rng(seed, cfg.config_id, "burst").permutation(T)[:n_hot]
        for t in hot:
            if not (idx[t] == 0).any():
                idx[t, 0] = 0
    return idx


def make_topk_weights(cfg: EPConfig, seed: int = 0) -> np.ndarray:
    logits = _rng(seed, cfg.config_id, "topk_weights").standard_normal((cfg.T, cfg.K))
    z = np.exp(logits - logits.max(axis=1, keepdims=True)) if cfg.T else logits
    w = z / z.sum(axis=1, keepdims=True) if cfg.T else z
    return np.ascontiguousarray(w, dtype=np.float32)


def _normal_bf16(rng: np.random.Generator, rows: int, H: int, chunk_rows: int = 4096) -> np.ndarray:
    out = np.empty((rows, H), dtype=np.uint16)
    for r0 in range(0, rows, chunk_rows):
        r1 = min(rows, r0 + chunk_rows)
        out[r0:r1] = to_bf16_bits(rng.standard_normal((r1 - r0, H), dtype=np.float32))
    return out


def make_x(cfg: EPConfig, seed: int = 0) -> np.ndarray:
    """Token activations as bf16 bit patterns, uint16 [T, H]."""
    return _normal_bf16(_rng(seed, cfg.config_id, "x"), cfg.T, cfg.H)


def make_out(cfg: EPConfig, rows: int, seed: int = 0) -> np.ndarray:
    """Synthetic expert outputs as bf16 bit patterns, uint16 [rows, H]."""
    return _normal_bf16(_rng(seed, cfg.config_id, "out"), rows, cfg.H)


def make_inputs(cfg: EPConfig, seed: int = 0, with_x: bool = True):
    d = {"topk_idx": make_topk_idx(cfg, seed), "topk_weights": make_topk_weights(cfg, seed)}
    if with_x:
        d["x"] = make_x(cfg, seed)
    return d


def shard_config(cfg: EPConfig, rank: int) -> EPConfig:
    """Replica `rank` of a multi-process run: same shapes, an independent seed stream."""
    return replace(cfg, config_id=cfg.config_id + 1000 * rank)
