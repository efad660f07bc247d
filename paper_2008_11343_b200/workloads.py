"""Seeded synthetic workloads: parameter-set shapes and per-worker gradients.

This module holds none of the method's arithmetic.  It only produces inputs
(parameter-set layouts, initial parameters, per-worker stochastic gradients)
and is the one module that both the CPU oracle's tests and the CUDA path's
tests and benchmark draw inputs from.

The paper trains BERT-Base (L=12, H=768, A=12, 110M parameters) and BERT-Large
(L=24, H=1024, A=16, 340M parameters) (Section 5.2, "Dataset and models"); the
datasets and trained models are not available, so only the *shapes* of those
parameter sets are reproduced and the gradients are random draws whose
per-tensor scale varies over several decades, as gradients of real layers do.

Every draw is a pure function of (SEED, config id, step, worker, tensor), so a
gradient can be regenerated anywhere (host for parity, device for throughput)
without storing it.  Host draws (numpy) and device draws (torch CUDA generator)
are different streams: parity tests always use the host stream and upload it.
"""
from __future__ import annotations

import dataclasses
import math
from typing import List, Optional, Sequence

import numpy as np

SEED = 200811343


@dataclasses.dataclass(frozen=True)
class Workload:
    """One synthetic configuration of the compressed-step benchmark."""

    name: str
    cfg_id: int
    n: int                      # simulated data-parallel workers
    chunk: int                  # compressor block length, elements
    tensor_sizes: tuple         # flat parameter vector = concatenation of these
    dist: str                   # "gauss" | "student_t3"
    scale_lo: float             # per-tensor gradient scale, log-uniform range
    scale_hi: float
    zero_frac: float = 0.0      # iid Bernoulli fraction of exactly-zero gradient entries
    x0_std: float = 0.02
    beta1: float = 0.9
    beta2: float = 0.999
    eps: float = 1e-8
    lr: float = 1e-4
    warmup_steps: int = 5
    compressed_steps: int = 10

    @property
    def d(self) -> int:
        return int(sum(self.tensor_sizes))

    @property
    def n_chunks(self) -> int:
        return (self.d + self.chunk - 1) // self.chunk

    @property
    def n_words(self) -> int:
        return (self.d + 31) // 32

    def tensor_offsets(self) -> np.ndarray:
        return np.concatenate([[0], np.cumsum(np.asarray(self.tensor_sizes, dtype=np.int64))])

    def tensor_scales(self) -> np.ndarray:
        """Per-tensor gradient scale, fixed for the whole run (log-uniform)."""
        rng = np.random.default_rng(np.random.SeedSequence([SEED, self.cfg_id, 0xA11CE]))
        u = rng.random(len(self.tensor_sizes))
        lo, hi = math.log(self.scale_lo), math.log(self.scale_hi)
        return np.exp(lo + (hi - lo) * u)

    def with_(self, **kw) -> "Workload":
        return dataclasses.replace(self, **kw)


def bert_tensor_sizes(layers: int, hidden: int, ffn: int, vocab: int = 30522,
                      max_pos: int = 512, type_vocab: int = 2) -> tuple:
    """Per-tensor element counts of a BERT encoder with pooler, in model order."""
    sizes: List[int] = [vocab * hidden, max_pos * hidden, type_vocab * hidden, hidden, hidden]
    for _ in range(layers):
        for _ in range(4):                      # Q, K, V, attention output
            sizes += [hidden * hidden, hidden]
        sizes += [hidden, hidden]               # LayerNorm
        sizes += [hidden * ffn, ffn]            # FFN in
        sizes += [ffn * hidden, hidden]         # FFN out
        sizes += [hidden, hidden]               # LayerNorm
    sizes += [hidden * hidden, hidden]          # pooler
    return tuple(sizes)


def _log_uniform_partition(total: int, parts: int, lo: int, hi: int, cfg_id: int) -> tuple:
    """`parts` sizes drawn log-uniform in [lo, hi], rescaled so they sum to `total`."""
    rng = np.random.default_rng(np.random.SeedSequence([SEED, cfg_id, 0x51235]))
    raw = np.exp(rng.uniform(math.log(lo), math.log(hi), size=parts))
    sizes = np.maximum(1, np.floor(raw * (total / raw.sum()))).astype(np.int64)
    sizes[-1] += total - int(sizes.sum())
    assert sizes[-1] > 0 and int(sizes.sum()) == total
    return tuple(int(s) for s in sizes)


def config(idx: int) -> Workload:
    """The benchmark configurations.

    0: one flat tensor, d = 2^20, n = 4, chunk = 4096 (fits in L2; parity-sized).
    1: d = 2^24 in 64 tensors of log-uniform size, 20 % zero gradients, n = 8.
    2: BERT-Base-shaped parameter set, n = 16, chunk = 16384.
    3: BERT-Large-shaped parameter set, n = 16, chunk = 32768, Student-t(3) gradients (headline).
    """
    if idx == 0:
        return Workload("flat-1M", 0, n=4, chunk=4096, tensor_sizes=(1 << 20,), dist="gauss",
                        scale_lo=0.01, scale_hi=0.01, warmup_steps=5, compressed_steps=10)
    if idx == 1:
        return Workload("mixed-16M", 1, n=8, chunk=8192,
                        tensor_sizes=_log_uniform_partition(1 << 24, 64, 4096, 1 << 20, 1),
                        dist="gauss", scale_lo=1e-4, scale_hi=1e-1, zero_frac=0.2,
                        warmup_steps=10, compressed_steps=50)
    if idx == 2:
        return Workload("bert-base", 2, n=16, chunk=16384,
                        tensor_sizes=bert_tensor_sizes(12, 768, 3072), dist="gauss",
                        scale_lo=1e-5, scale_hi=1e-2, warmup_steps=5, compressed_steps=20)
    if idx == 3:
        return Workload("bert-large", 3, n=16, chunk=32768,
                        tensor_sizes=bert_tensor_sizes(24, 1024, 4096), dist="student_t3",
                        scale_lo=1e-5, scale_hi=1e-2, warmup_steps=5, compressed_steps=20)
    raise ValueError(f"unknown config index {idx}")


def sliced(w: Workload, d: int, name: Optional[str] = None) -> Workload:
    """The first `d` elements of a workload's flat vector (a bounded sample of it)."""
    sizes, left = [], d
    for s in w.tensor_sizes:
        if left <= 0:
            break
        sizes.append(min(s, left))
        left -= sizes[-1]
    assert left == 0, "slice longer than the workload"
    return w.with_(tensor_sizes=tuple(sizes), name=name or f"{w.name}[:{d}]")


# --------------------------------------------------------------------------- host draws

def _rng(w: Workload, *key: int) -> np.random.Generator:
    return np.random.default_rng(np.random.SeedSequence([SEED, w.cfg_id, *key]))


def initial_params(w: Workload) -> np.ndarray:
    return (_rng(w, 0x0A) .standard_normal(w.d, dtype=np.float32) * np.float32(w.x0_std))


def _unit_draw(rng: np.random.Generator, size: int, dist: str) -> np.ndarray:
    if dist == "gauss":
        return rng.standard_normal(size, dtype=np.float32)
    if dist == "student_t3":
        z = rng.standard_normal(size, dtype=np.float32)
        chi = rng.standard_normal((3, size), dtype=np.float32)
        den = np.sqrt((chi * chi).sum(axis=0) / np.float32(3.0))
        return (z / den).astype(np.float32)
    raise ValueError(dist)


def host_gradient(w: Workload, step: int, worker: int) -> np.ndarray:
    """Worker `worker`'s stochastic gradient at global step `step` (float32[d])."""
    out = np.empty(w.d, dtype=np.float32)
    offs, scales = w.tensor_offsets(), w.tensor_scales()
    for k, sz in enumerate(w.tensor_sizes):
        rng = _rng(w, 0x6, step, worker, k)
        g = _unit_draw(rng, sz, w.dist) * np.float32(scales[k])
        if w.zero_frac > 0.0:
            g[rng.random(sz, dtype=np.float32) < w.zero_frac] = 0.0
        out[offs[k]:offs[k + 1]] = g
    return out


def host_gradients(w: Workload, step: int) -> List[np.ndarray]:
    return [host_gradient(w, step, i) for i in range(w.n)]


# --------------------------------------------------------------------------- device draws

def device_gradient(w: Workload, step: int, worker: int, out, piece: int = 1 << 24) -> None:
    """Fill the CUDA float32 tensor `out` (d elements) with a gradient draw.

    Same distribution family as `host_gradient`, different random stream (the
    torch CUDA generator); used only where throughput is measured.
    """
    import torch

    gen = torch.Generator(device=out.device)
    gen.manual_seed((SEED * 1000003 + w.cfg_id * 7919 + step * 104729 + worker) & 0x7FFFFFFFFFFF)
    offs, scales = w.tensor_offsets(), w.tensor_scales()
    for k, sz in enumerate(w.tensor_sizes):
        for a in range(0, sz, piece):
            b = min(sz, a + piece)
            view = out[offs[k] + a: offs[k] + b]
            view.normal_(0.0, 1.0, generator=gen)
            if w.dist == "student_t3":
                chi = torch.empty((3, b - a), dtype=torch.float32, device=out.device)
                chi.normal_(0.0, 1.0, generator=gen)
                view.div_(chi.square_().sum(dim=0).div_(3.0).sqrt_())
            view.mul_(float(scales[k]))
            if w.zero_frac > 0.0:
                mask = torch.empty(b - a, dtype=torch.float32, device=out.device)
                mask.uniform_(0.0, 1.0, generator=gen)
                view.masked_fill_(mask < w.zero_frac, 0.0)


def sample_chunks(w: Workload, how_many: int, seed_key: int = 0) -> Sequence[int]:
    """Chunk indices for sampled full-size parity: first, last (ragged) and random ones."""
    C = w.n_chunks
    picks = {0, C - 1}
    rng = _rng(w, 0xC4, seed_key)
    while len(picks) < min(how_many, C):
        picks.add(int(rng.integers(0, C)))
    return sorted(picks)
