"""Seeded synthetic inputs for the VScan reduction path.

These arrays stand in for what a LLaVA / Qwen-VL forward pass would hand to the
reduction steps (Sec. 4.1, 4.2): encoder features, per-head [CLS] attention
rows of two encoder layers, and the query / key / value / hidden tensors of one
LLM layer.  The module holds no arithmetic of the method itself: it only draws
numbers with the stated distributions, so both the CPU oracle's tests and the
CUDA path's tests can start from identical inputs.

Every tensor is returned as a float32 numpy array whose values are exactly
representable in the workload's I/O dtype (bf16 values are rounded to nearest
even first), so a later cast to that dtype is lossless.

RNG: one numpy Philox stream per (seed, config id, tensor, instance); the first
n instances of a batch are therefore the same whatever the batch size.
"""
from __future__ import annotations

from concurrent.futures import ThreadPoolExecutor
import os

import numpy as np
import torch

from .configs import VScanConfig

_TENSOR_IDS = {"x": 1, "attn_g": 2, "attn_l": 3, "q_last": 4, "k": 5, "v": 6, "hidden": 7,
               "redraw": 8}


def rng_for(seed: int, cfg: VScanConfig, tensor: str, instance: int, sub: int = 0) -> np.random.Generator:
    key = (int(seed) << 96) | (int(cfg.config_id) << 80) | (int(sub) << 40) \
        | (_TENSOR_IDS[tensor] << 32) | int(instance)
    return np.random.Generator(np.random.Philox(key=key))


def round_to_dtype(a: np.ndarray, dtype: str) -> np.ndarray:
    """float32 array whose values are representable in `dtype` (round to nearest even)."""
    a = np.ascontiguousarray(a, dtype=np.float32)
    if dtype == "f32":
        return a
    if dtype == "bf16":
        return torch.from_numpy(a).to(torch.bfloat16).to(torch.float32).numpy()
    raise ValueError(dtype)


def _pmap(fn, n):
    workers = min(n, os.cpu_count() or 1, 16)
    if workers <= 1:
        return [fn(i) for i in range(n)]
    with ThreadPoolExecutor(workers) as ex:
        return list(ex.map(fn, range(n)))


def features_one(cfg: VScanConfig, seed: int, inst: int) -> np.ndarray:
    """[L, D] features: cluster centres ~ N(0, I), token = centre + 0.3 N(0, I)."""
    g = rng_for(seed, cfg, "x", inst)
    centres = g.standard_normal((cfg.n_clusters, cfg.D), dtype=np.float32)
    cid = g.integers(0, cfg.n_clusters, size=cfg.L)
    x = centres[cid] + np.float32(0.3) * g.standard_normal((cfg.L, cfg.D), dtype=np.float32)
    return round_to_dtype(x, cfg.dtype)


def redraw_token(cfg: VScanConfig, seed: int, inst: int, token_row: int, x_inst: np.ndarray,
                 attempt: int) -> np.ndarray:
    """A fresh noise draw of the same scale for one feature row (keeps the row's old mean)."""
    g = rng_for(seed, cfg, "redraw", inst, sub=(token_row << 8) | (attempt & 0xFF))
    old = x_inst[token_row]
    noise = np.float32(0.3) * g.standard_normal(cfg.D, dtype=np.float32)
    # move the row by a fresh perturbation of the generator's noise scale
    return round_to_dtype(old + np.float32(0.5) * noise, cfg.dtype)


def attention_rows_one(cfg: VScanConfig, seed: int, inst: int, which: str) -> np.ndarray:
    """[H, L] rows of probabilities: softmax over L of 3 * N(0,1) logits, per head."""
    g = rng_for(seed, cfg, which, inst)
    z = 3.0 * g.standard_normal((cfg.H, cfg.L))
    z -= z.max(axis=1, keepdims=True)
    p = np.exp(z)
    p /= p.sum(axis=1, keepdims=True)
    return round_to_dtype(p.astype(np.float32), cfg.dtype)


def stage1_inputs(cfg: VScanConfig, seed: int = 0, instances: int | None = None) -> dict:
    n = cfg.instances if instances is None else instances
    x = np.stack(_pmap(lambda i: features_one(cfg, seed, i), n))
    ag = np.stack(_pmap(lambda i: attention_rows_one(cfg, seed, i, "attn_g"), n))
    al = np.stack(_pmap(lambda i: attention_rows_one(cfg, seed, i, "attn_l"), n))
    return {"x": x, "attn_g": ag, "attn_l": al}


def stage2_inputs(cfg: VScanConfig, seed: int = 0, batch: int | None = None) -> dict:
    """q_last [B,Hq,d], k/v [B,Hkv,S,d] ~ N(0, sigma=1/sqrt(d)); hidden [B,S,Dh] ~ N(0,1);
    pos_ids [P,B,S] = 0..S-1 on every plane; scale = 1/sqrt(d)."""
    n = cfg.B if batch is None else batch
    sigma = np.float32(1.0 / np.sqrt(cfg.d))

    def one(b):
        q = sigma * rng_for(seed, cfg, "q_last", b).standard_normal((cfg.Hq, cfg.d), dtype=np.float32)
        k = sigma * rng_for(seed, cfg, "k", b).standard_normal((cfg.Hkv, cfg.S, cfg.d), dtype=np.float32)
        v = sigma * rng_for(seed, cfg, "v", b).standard_normal((cfg.Hkv, cfg.S, cfg.d), dtype=np.float32)
        h = rng_for(seed, cfg, "hidden", b).standard_normal((cfg.S, cfg.Dh), dtype=np.float32)
        return (round_to_dtype(q, cfg.dtype), round_to_dtype(k, cfg.dtype),
                round_to_dtype(v, cfg.dtype), round_to_dtype(h, cfg.dtype))

    parts = _pmap(one, n)
    pos = np.broadcast_to(np.arange(cfg.S, dtype=np.int32), (cfg.pos_planes, n, cfg.S)).copy()
    return {"q_last": np.stack([p[0] for p in parts]), "k": np.stack([p[1] for p in parts]),
            "v": np.stack([p[2] for p in parts]), "hidden": np.stack([p[3] for p in parts]),
            "pos_ids": pos, "scale": float(1.0 / np.sqrt(cfg.d))}
