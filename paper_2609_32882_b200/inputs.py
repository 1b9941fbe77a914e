"""Seeded synthetic inputs for the VSA2 attention path.

This module holds no arithmetic of the method: it only draws random tensors with
the shapes and the spatio-temporal structure of video-DiT activations and casts
them to bf16 bit patterns.  Both the CUDA path's tests/benchmark and the CPU
oracle's tests are fed from here, so that the two see identical bits.

Recipes (every stream is numpy's PCG64 seeded with [seed, tensor id, batch, head],
so any single head can be regenerated without the others):

* "iid":      x ~ N(0, 1) per element.
* "locality": white N(0,1) noise on the (t, h, w) grid per channel, smoothed with a
              separable Gaussian filter (sigma = 2 tokens along t, h and w, reflect
              boundary, truncated at 4 sigma), rescaled to unit standard deviation
              over the head, plus 0.3 * N(0, 1) per element.
* gate:       constant, or tanh(N(0, 0.5^2)) per token per head.
* dO:         N(0, 1) per element, bf16.

These stand in for the private video latents of the paper's runs.
"""
from __future__ import annotations

import dataclasses
from concurrent.futures import ThreadPoolExecutor

import numpy as np

PER_SEQUENCE, PER_QUERY, PER_QUERY_BUDGET = 0, 1, 2
_TENSOR_ID = {"q": 0, "k": 1, "v": 2, "do": 3, "gate": 4, "budget": 5}


@dataclasses.dataclass(frozen=True)
class Workload:
    name: str
    batch: int
    heads_q: int
    heads_kv: int
    head_dim: int
    grid: tuple          # (t, h, w) valid latent grid
    cube: tuple = (4, 4, 4)
    rpool: tuple = (2, 2, 2)
    select_mode: int = PER_SEQUENCE
    topk: int = 0
    kind: str = "locality"
    seed: int = 0
    gate_const: float | None = None
    text_len: int = 0    # text tokens appended to every head's token rows (MMDiT joint attention)

    @property
    def L(self):
        return self.grid[0] * self.grid[1] * self.grid[2]

    @property
    def n_cubes(self):
        return int(np.prod([-(-g // c) for g, c in zip(self.grid, self.cube)]))

    def replace(self, **kw):
        return dataclasses.replace(self, **kw)


# The five configurations of the build's baseline file (index = config number).
CONFIGS = {
    0: Workload("tiny", 1, 2, 2, 64, (4, 8, 8), select_mode=PER_QUERY, topk=2, kind="iid", seed=0, gate_const=0.5),
    1: Workload("small_video", 1, 12, 12, 128, (8, 16, 16), select_mode=PER_QUERY, topk=8, seed=1),
    2: Workload("480p", 1, 12, 3, 128, (21, 30, 52), select_mode=PER_QUERY, topk=78, seed=2),
    3: Workload("720p_top64", 1, 40, 40, 128, (21, 45, 80), select_mode=PER_SEQUENCE, topk=64, seed=3),
    4: Workload("720p_sweep", 1, 40, 40, 128, (21, 45, 80), select_mode=PER_QUERY_BUDGET, topk=0, seed=4),
}


def f32_to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """float32 -> bf16 bit patterns (uint16), round to nearest even."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    lsb = (u >> np.uint32(16)) & np.uint32(1)
    return ((u + np.uint32(0x7FFF) + lsb) >> np.uint32(16)).astype(np.uint16)


def bf16_bits_to_f32(bits: np.ndarray) -> np.ndarray:
    return (np.ascontiguousarray(bits, dtype=np.uint16).astype(np.uint32) << np.uint32(16)).view(np.float32)


def _rng(seed, name, b, h):
    return np.random.default_rng([int(seed), _TENSOR_ID[name], int(b), int(h)])


def head_tensor(wl: Workload, name: str, b: int, h: int) -> np.ndarray:
    """One head of q, k, v or do as bf16 bit patterns, shape [L + text_len, D]: the video tokens in raster order, then the
    text tokens (i.i.d. N(0,1): text embeddings carry no spatial structure)."""
    x = _head_video(wl, name, b, h)
    if wl.text_len:
        rng = np.random.default_rng([int(wl.seed), _TENSOR_ID[name], int(b), int(h), 7])
        x = np.concatenate([x, f32_to_bf16_bits(rng.standard_normal((wl.text_len, wl.head_dim), dtype=np.float32))])
    return x


def _head_video(wl: Workload, name: str, b: int, h: int) -> np.ndarray:
    rng = _rng(wl.seed, name, b, h)
    t, hh, w = wl.grid
    d = wl.head_dim
    if wl.kind == "iid" or name == "do":
        x = rng.standard_normal((wl.L, d), dtype=np.float32)
    elif wl.kind == "locality":
        from scipy.ndimage import gaussian_filter
        white = rng.standard_normal((t, hh, w, d), dtype=np.float32)
        smooth = gaussian_filter(white, sigma=(2.0, 2.0, 2.0, 0.0), mode="reflect", truncate=4.0)
        smooth /= smooth.std()
        x = (smooth + np.float32(0.3) * rng.standard_normal((t, hh, w, d), dtype=np.float32)).reshape(wl.L, d)
    else:
        raise ValueError(wl.kind)
    return f32_to_bf16_bits(x)


def head_gate(wl: Workload, b: int, h: int) -> np.ndarray:
    """Gate values of one query head, float32 [L]."""
    if wl.gate_const is not None:
        return np.full(wl.L, wl.gate_const, dtype=np.float32)
    rng = _rng(wl.seed, "gate", b, h)
    return np.tanh(np.float32(0.5) * rng.standard_normal(wl.L, dtype=np.float32)).astype(np.float32)


def head_budgets(wl: Workload, b: int, h: int, lo=16, hi=256) -> np.ndarray:
    """Per-query-block KV budgets of one head, int32 [N], uniform in [lo, hi]."""
    rng = _rng(wl.seed, "budget", b, h)
    return rng.integers(lo, hi + 1, size=wl.n_cubes, dtype=np.int32)


def _stack(fn, nb, nh, threads):
    jobs = [(b, h) for b in range(nb) for h in range(nh)]
    if threads > 1 and len(jobs) > 1:
        with ThreadPoolExecutor(threads) as ex:
            parts = list(ex.map(lambda bh: fn(*bh), jobs))
    else:
        parts = [fn(*bh) for bh in jobs]
    return np.stack(parts).reshape((nb, nh) + parts[0].shape)


def make_inputs(wl: Workload, with_grad=True, threads=8) -> dict:
    """All tensors of a workload: q [B,Hq,L,D], k, v [B,Hkv,L,D] (uint16 bf16 bits),
    gate [B,Hq,L] float32 and, if asked, do [B,Hq,L,D] (uint16 bf16 bits)."""
    out = {
        "q": _stack(lambda b, h: head_tensor(wl, "q", b, h), wl.batch, wl.heads_q, threads),
        "k": _stack(lambda b, h: head_tensor(wl, "k", b, h), wl.batch, wl.heads_kv, threads),
        "v": _stack(lambda b, h: head_tensor(wl, "v", b, h), wl.batch, wl.heads_kv, threads),
        "gate": _stack(lambda b, h: head_gate(wl, b, h), wl.batch, wl.heads_q, threads),
    }
    if with_grad:
        out["do"] = _stack(lambda b, h: head_tensor(wl, "do", b, h), wl.batch, wl.heads_q, threads)
    if wl.select_mode == PER_QUERY_BUDGET:
        out["budgets"] = _stack(lambda b, h: head_budgets(wl, b, h), wl.batch, wl.heads_q, 1)
    return out
