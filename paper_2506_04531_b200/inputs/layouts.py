"""Synthetic parameter layouts shaped like the decoder-only LLMs the paper trains (Pythia-70M,
-160M, -410M in its evaluation section) plus a 1.4B-class layout for the bandwidth sweep.

A layout is an ordered list of tensors packed back to back in one flat fp32 buffer:
embed_in, then per layer {ln1.w, ln1.b, qkv.w, qkv.b, attn_out.w, attn_out.b, ln2.w, ln2.b,
up.w, up.b, down.w, down.b}, then final_ln.w, final_ln.b, embed_out (untied).
P = 2*V*d + layers*(12 d^2 + 13 d) + 2 d ; tensors = 4 + 12*layers.

This module holds shapes only: none of the method's arithmetic.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import List, Tuple

import numpy as np

KIND_MATRIX, KIND_NORM_WEIGHT, KIND_BIAS = 0, 1, 2


@dataclass(frozen=True)
class Tensor:
    name: str
    shape: Tuple[int, ...]
    kind: int

    @property
    def numel(self) -> int:
        n = 1
        for s in self.shape:
            n *= s
        return n


@dataclass(frozen=True)
class Layout:
    name: str
    tensors: Tuple[Tensor, ...]

    @property
    def numel(self) -> np.ndarray:
        return np.array([t.numel for t in self.tensors], dtype=np.uint64)

    @property
    def offsets(self) -> np.ndarray:
        """Exclusive prefix sum of tensor sizes, length n_tensors + 1."""
        return np.concatenate([[0], np.cumsum(self.numel)]).astype(np.uint64)

    @property
    def P(self) -> int:
        return int(self.numel.sum())

    @property
    def n_tensors(self) -> int:
        return len(self.tensors)

    def per_tensor(self, matrix: float, norm_weight: float, bias: float) -> np.ndarray:
        """A float32 value per tensor chosen by tensor kind."""
        pick = {KIND_MATRIX: matrix, KIND_NORM_WEIGHT: norm_weight, KIND_BIAS: bias}
        return np.array([pick[t.kind] for t in self.tensors], dtype=np.float32)


def decoder_layout(name: str, layers: int, d: int, vocab: int) -> Layout:
    ts: List[Tensor] = [Tensor("embed_in", (vocab, d), KIND_MATRIX)]
    for i in range(layers):
        p = f"layers.{i}."
        ts += [
            Tensor(p + "ln1.w", (d,), KIND_NORM_WEIGHT), Tensor(p + "ln1.b", (d,), KIND_BIAS),
            Tensor(p + "qkv.w", (3 * d, d), KIND_MATRIX), Tensor(p + "qkv.b", (3 * d,), KIND_BIAS),
            Tensor(p + "attn_out.w", (d, d), KIND_MATRIX), Tensor(p + "attn_out.b", (d,), KIND_BIAS),
            Tensor(p + "ln2.w", (d,), KIND_NORM_WEIGHT), Tensor(p + "ln2.b", (d,), KIND_BIAS),
            Tensor(p + "up.w", (4 * d, d), KIND_MATRIX), Tensor(p + "up.b", (4 * d,), KIND_BIAS),
            Tensor(p + "down.w", (d, 4 * d), KIND_MATRIX), Tensor(p + "down.b", (d,), KIND_BIAS),
        ]
    ts += [Tensor("final_ln.w", (d,), KIND_NORM_WEIGHT), Tensor("final_ln.b", (d,), KIND_BIAS),
           Tensor("embed_out", (vocab, d), KIND_MATRIX)]
    return Layout(name, tuple(ts))


def flat_layout(name: str, P: int) -> Layout:
    return Layout(name, (Tensor("flat", (int(P),), KIND_MATRIX),))


def ragged_layout(name: str, sizes) -> Layout:
    """Tensors of arbitrary (odd) lengths, alternating kinds; used by edge-case tests."""
    kinds = (KIND_MATRIX, KIND_NORM_WEIGHT, KIND_BIAS)
    return Layout(name, tuple(Tensor(f"t{i}", (int(n),), kinds[i % 3]) for i, n in enumerate(sizes)))


def named_layout(name: str) -> Layout:
    if name == "toy":
        return flat_layout("toy", 1 << 20)
    if name == "70m":
        return decoder_layout("70m", 6, 512, 50304)
    if name == "160m":
        return decoder_layout("160m", 12, 768, 50304)
    if name == "410m":
        return decoder_layout("410m", 24, 1024, 50304)
    if name == "1p4b":
        return decoder_layout("1p4b", 24, 2048, 50304)
    raise KeyError(name)
