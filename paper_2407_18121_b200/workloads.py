"""Seeded synthetic inputs shaped like LLaVA-1.5 prompts and decode steps.

This module only draws random tensors and rounds them to bf16. It contains none
of the cache-merging arithmetic, so both the CUDA path and the CPU oracle can be
fed from it without sharing any of the method's code.

Every tensor is returned as a numpy ``uint16`` array holding bf16 bit patterns.
A problem index ``n`` enumerates (batch element, layer) pairs, ``n = b * layers + l``;
each ``n`` has its own counter-seeded generator, so any subset of problems can be
drawn without drawing the others and chunks can be produced in parallel.
"""
from __future__ import annotations

import dataclasses
import math
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass
from typing import Iterable, Sequence, Tuple

import numpy as np

_PROMPT_STREAM = 0
_DECODE_STREAM = 1


@dataclass(frozen=True)
class Workload:
    """Shape and recipe of one synthetic configuration."""
    name: str
    batch: int
    layers: int
    heads: int
    head_dim: int
    prompt_len: int
    keep_ratios: Tuple[float, ...]
    decode_steps: int
    scale: float
    offset: int
    seed: int
    kind: str            # "peaked" | "lowrank" | "zipf"
    n_image: int = 0     # leading positions that carry the redundant component
    rank: int = 0        # rank of that component

    @property
    def N(self) -> int:
        return self.batch * self.layers

    @property
    def keep_ratio(self) -> float:
        return self.keep_ratios[0]

    def shrunk(self, batch: int | None = None, layers: int | None = None,
               decode_steps: int | None = None) -> "Workload":
        """Same recipe with fewer problems / steps (problem n keeps its draws only
        when ``layers`` is unchanged, because n = b * layers + l)."""
        return dataclasses.replace(
            self,
            batch=self.batch if batch is None else batch,
            layers=self.layers if layers is None else layers,
            decode_steps=self.decode_steps if decode_steps is None else decode_steps,
        )


WORKLOADS = {
    # tiny single-layer case, peaked attention
    "tiny": Workload("tiny", 1, 1, 8, 64, 256, (0.5,), 32, 1.0, 16, 0, "peaked", n_image=128),
    # LLaVA-1.5-7B shapes, batch 1, 576 image + 64 text tokens
    "llava7b_b1": Workload("llava7b_b1", 1, 32, 32, 128, 640, (0.5,), 512,
                           1.0 / math.sqrt(128.0), 16, 1, "lowrank", n_image=576, rank=8),
    # same shapes, batch 8, 576 image + 448 text tokens
    "llava7b_b8": Workload("llava7b_b8", 8, 32, 32, 128, 1024, (0.25,), 512,
                           1.0 / math.sqrt(128.0), 16, 2, "lowrank", n_image=576, rank=8),
    # LLaVA-1.5-13B shapes, batch 4, 1704 image + 344 text tokens, ratio sweep
    "llava13b_b4": Workload("llava13b_b4", 4, 40, 40, 128, 2048, (0.1, 0.25, 0.5, 0.75), 1024,
                            1.0 / math.sqrt(128.0), 16, 3, "lowrank", n_image=1704, rank=16),
    # long-context stress, heavy-tailed importance
    "long8k": Workload("long8k", 16, 4, 32, 128, 8192, (0.1,), 2048,
                       1.0 / math.sqrt(128.0), 16, 4, "zipf"),
    # Qwen-VL-7B shapes (Sec. 4.1 names it as the second backbone): 32 layers x 32 heads x 128, 256 image
    # tokens (its adapter's fixed output length) + 64 text tokens, the paper's recent distance of 25.
    # Not one of the five measured configurations: an extra parity and timing case.
    "qwenvl7b_b1": Workload("qwenvl7b_b1", 1, 32, 32, 128, 320, (0.5,), 512,
                            1.0 / math.sqrt(128.0), 25, 5, "lowrank", n_image=256, rank=8),
}
CONFIG_ORDER = ("tiny", "llava7b_b1", "llava7b_b8", "llava13b_b4", "long8k")


def to_bf16_bits(x: np.ndarray) -> np.ndarray:
    """Round fp32 to bf16 (round to nearest, ties to even); returns uint16 bit patterns."""
    u = np.ascontiguousarray(x, dtype=np.float32).view(np.uint32)
    r = (u + (np.uint32(0x7FFF) + ((u >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return r.astype(np.uint16)


def bf16_bits_to_f64(b: np.ndarray) -> np.ndarray:
    """Widen bf16 bit patterns exactly to float64."""
    u = b.astype(np.uint32) << np.uint32(16)
    return u.view(np.float32).astype(np.float64)


def _rng(seed: int, stream: int, index: int) -> np.random.Generator:
    return np.random.Generator(np.random.PCG64(np.random.SeedSequence([seed, stream, index])))


def prompt_problem(w: Workload, n: int):
    """Q, K, V of problem ``n``: three uint16 arrays of shape [H, T, D] (bf16 bits)."""
    H, T, D = w.heads, w.prompt_len, w.head_dim
    g = _rng(w.seed, _PROMPT_STREAM, n)
    Q = g.standard_normal((H, T, D), dtype=np.float32)
    K = g.standard_normal((H, T, D), dtype=np.float32)
    V = g.standard_normal((H, T, D), dtype=np.float32)
    if w.kind == "peaked":
        # keys shrunk by 1/sqrt(D); four boosted key positions per head along one shared direction
        K *= np.float32(1.0 / math.sqrt(D))
        u = g.standard_normal(D, dtype=np.float32)
        u /= np.linalg.norm(u)
        for h in range(H):
            pos = g.choice(T, size=4, replace=False)
            K[h, pos, :] += np.float32(3.0) * u
    elif w.kind == "lowrank":
        # image tokens share a rank-r component across heads and across K / V
        r, ni = w.rank, w.n_image
        a = g.standard_normal((ni, r), dtype=np.float32)
        WK = g.standard_normal((H, r, D), dtype=np.float32) * np.float32(2.0 / math.sqrt(r))
        WV = g.standard_normal((H, r, D), dtype=np.float32) * np.float32(2.0 / math.sqrt(r))
        K[:, :ni, :] += np.einsum("tr,hrd->htd", a, WK)
        V[:, :ni, :] += np.einsum("tr,hrd->htd", a, WV)
    elif w.kind == "zipf":
        # one shared direction whose weight over positions follows rank^-1.1
        u = g.standard_normal(D, dtype=np.float32)
        u /= np.linalg.norm(u)
        rank = g.permutation(T).astype(np.float32) + np.float32(1.0)
        wt = rank ** np.float32(-1.1)
        K += (np.float32(6.0) * wt)[None, :, None] * u[None, None, :]
        Q += np.float32(math.sqrt(D)) * u[None, None, :]
    else:
        raise ValueError(f"unknown workload kind {w.kind!r}")
    return to_bf16_bits(Q), to_bf16_bits(K), to_bf16_bits(V)


def prompt(w: Workload, problems: Iterable[int] | None = None, threads: int = 8):
    """Q, K, V for the listed problems (default: all), each [len(problems), H, T, D] uint16."""
    idx = list(range(w.N)) if problems is None else list(problems)
    shape = (len(idx), w.heads, w.prompt_len, w.head_dim)
    Q = np.empty(shape, np.uint16)
    K = np.empty(shape, np.uint16)
    V = np.empty(shape, np.uint16)

    def fill(i):
        Q[i], K[i], V[i] = prompt_problem(w, idx[i])

    if len(idx) > 1 and threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(len(idx))))
    else:
        for i in range(len(idx)):
            fill(i)
    return Q, K, V


def decode_step_inputs(w: Workload, step: int, problems: Sequence[int] | None = None):
    """q, k_new, v_new of one decode step: uint16 [N, H, D] (or the listed problems' rows)."""
    g = _rng(w.seed, _DECODE_STREAM, step)
    shape = (w.N, w.heads, w.head_dim)
    q = g.standard_normal(shape, dtype=np.float32)
    k = g.standard_normal(shape, dtype=np.float32)
    v = g.standard_normal(shape, dtype=np.float32)
    if w.kind == "peaked":
        k *= np.float32(1.0 / math.sqrt(w.head_dim))
    if problems is not None:
        sel = np.asarray(list(problems), dtype=np.int64)
        q, k, v = q[sel], k[sel], v[sel]
    return to_bf16_bits(q), to_bf16_bits(k), to_bf16_bits(v)


def decode_inputs(w: Workload, steps: int | None = None, problems: Sequence[int] | None = None,
                  threads: int = 8):
    """All decode steps stacked: three uint16 arrays [steps, N, H, D]."""
    S = w.decode_steps if steps is None else steps
    n = w.N if problems is None else len(list(problems))
    shape = (S, n, w.heads, w.head_dim)
    q = np.empty(shape, np.uint16)
    k = np.empty(shape, np.uint16)
    v = np.empty(shape, np.uint16)

    def fill(s):
        q[s], k[s], v[s] = decode_step_inputs(w, s, problems)

    if S > 1 and threads > 1:
        with ThreadPoolExecutor(max_workers=threads) as ex:
            list(ex.map(fill, range(S)))
    else:
        for s in range(S):
            fill(s)
    return q, k, v
