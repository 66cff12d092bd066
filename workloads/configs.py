"""The five synthetic workloads and their seeded inputs.

Each workload fixes the number of simulated workers K, the tensor sizes of the flat
parameter set, the optimiser constants, the number of rounds T and how gradients are
drawn from the counter hash.  Tensor sizes only mimic the *shape statistics* of the
model families they are named after (tensor count, size range, a few dominant
tensors); no dataset or model file is involved.

This module holds inputs and data layout only, none of the update/merge arithmetic.
"""
from __future__ import annotations

import json
import math
import os
from dataclasses import dataclass, field
from typing import List, Optional, Tuple

import numpy as np

from . import hashgen

_HERE = os.path.dirname(os.path.abspath(__file__))
ALIGN_ELEMS = 32            # every tensor starts on a 32-element (128-byte) boundary
SIZE_LO, SIZE_HI = 64, 2_400_000


# --------------------------------------------------------------------------- layout
def draw_log_uniform_sizes(seed: int, n: int, total: int, first_tensor: int = 0) -> List[int]:
    """n tensor sizes, log-uniform in [64, 2.4M], summing exactly to ``total``.

    raw_t = exp(ln 64 + u_t (ln 2.4e6 - ln 64)) with u_t from hash stream 3; a common
    scale factor (found by bisection) and a clamp to the size range bring the sum just
    below ``total``; the remainder is handed out in descending size order without
    exceeding the cap.
    """
    lo, hi = math.log(SIZE_LO), math.log(SIZE_HI)
    raw = [math.exp(lo + hashgen.layout_u(seed, first_tensor + t) * (hi - lo)) for t in range(n)]

    def sizes_at(scale: float) -> List[int]:
        return [min(SIZE_HI, max(SIZE_LO, int(scale * x))) for x in raw]

    a, b = 0.0, 1.0
    while sum(sizes_at(b)) <= total and b < 1e9:
        b *= 2.0
    for _ in range(200):
        mid = 0.5 * (a + b)
        if sum(sizes_at(mid)) <= total:
            a = mid
        else:
            b = mid
    sizes = sizes_at(a)
    rest = total - sum(sizes)
    if rest < 0:
        raise ValueError("total too small for %d tensors" % n)
    for t in sorted(range(n), key=lambda t: (-sizes[t], t)):
        add = min(rest, SIZE_HI - sizes[t])
        sizes[t] += add
        rest -= add
        if rest == 0:
            break
    if rest:
        raise ValueError("total too large for %d tensors" % n)
    return sizes


class Layout:
    """Offsets of the tensors inside the flat, padded buffers."""

    def __init__(self, sizes: List[int]):
        self.sizes = [int(s) for s in sizes]
        self.offsets = []            # start of tensor t in the padded buffer
        self.starts = []             # start of tensor t in the un-padded concatenation
        pos = 0
        flat = 0
        for s in self.sizes:
            self.offsets.append(pos)
            self.starts.append(flat)
            pos += -(-s // ALIGN_ELEMS) * ALIGN_ELEMS
            flat += s
        self.P = flat
        self.P_pad = pos

    def pack(self, flat: np.ndarray) -> np.ndarray:
        """Un-padded concatenation -> padded buffer (pads are zero)."""
        out = np.zeros(self.P_pad, dtype=flat.dtype)
        for s, o, f in zip(self.sizes, self.offsets, self.starts):
            out[o:o + s] = flat[f:f + s]
        return out

    def unpack(self, padded: np.ndarray) -> np.ndarray:
        """Padded buffer -> un-padded concatenation."""
        out = np.empty(self.P, dtype=padded.dtype)
        for s, o, f in zip(self.sizes, self.offsets, self.starts):
            out[f:f + s] = padded[o:o + s]
        return out

    def padded_index(self, flat_idx: np.ndarray) -> np.ndarray:
        """Map indices of the un-padded concatenation to positions in the padded buffer."""
        starts = np.asarray(self.starts, dtype=np.int64)
        offs = np.asarray(self.offsets, dtype=np.int64)
        t = np.searchsorted(starts, flat_idx, side="right") - 1
        return offs[t] + (np.asarray(flat_idx, dtype=np.int64) - starts[t])


# --------------------------------------------------------------------------- configs
@dataclass(frozen=True)
class Workload:
    name: str
    K: int
    sizes: Tuple[int, ...]
    T: int
    lr: float
    momentum: float
    weight_decay: float
    seed: int
    grad_kind: str                 # "uniform" (scale * U[-1,1)) or "gauss" (N(0, sigma))
    grad_scale: float              # scale or sigma
    grad_dtype: str = "f32"        # "f32" or "bf16" (storage of the gradient only)
    staleness: int = 1
    sparse: Optional[Tuple[int, int, int]] = None   # (tensor_id, rows, cols) of the embedding
    note: str = ""
    layout: Layout = field(init=False, compare=False, repr=False)

    def __post_init__(self):
        object.__setattr__(self, "layout", Layout(list(self.sizes)))

    @property
    def P(self) -> int:
        return self.layout.P

    # ---- seeded inputs (un-padded index space) -------------------------------------
    def initial_global(self, idx: Optional[np.ndarray] = None) -> np.ndarray:
        if idx is None:
            return hashgen.init_global(self.seed, idx0=0, n=self.P)
        return hashgen.init_global(self.seed, idx=idx)

    def sparse_rows(self, worker: int, step: int) -> np.ndarray:
        """Ascending int32 indices of the embedding rows with a gradient."""
        assert self.sparse is not None
        _, rows, _ = self.sparse
        return np.nonzero(hashgen.row_mask(self.seed, step, worker, rows))[0].astype(np.int32)

    def gradient(self, worker: int, step: int, idx: Optional[np.ndarray] = None) -> np.ndarray:
        """fp32 gradient of ``worker`` at round ``step`` before any storage rounding.

        Over the whole un-padded index space, or at the listed indices.  For a workload
        with a sparse-row embedding the rows without a gradient are zero.
        """
        if self.grad_kind == "uniform":
            gen = lambda **kw: hashgen.grad_uniform(self.seed, step, worker, scale=self.grad_scale, **kw)
        else:
            gen = lambda **kw: hashgen.grad_gauss(self.seed, step, worker, sigma=self.grad_scale, **kw)
        g = gen(idx0=0, n=self.P) if idx is None else gen(idx=idx)
        if self.sparse is not None:
            tid, rows, cols = self.sparse
            start = self.layout.starts[tid]
            active = hashgen.row_mask(self.seed, step, worker, rows)
            if idx is None:
                seg = g[start:start + rows * cols].reshape(rows, cols)
                seg[~active] = 0.0
            else:
                idx = np.asarray(idx, dtype=np.int64)
                inside = (idx >= start) & (idx < start + rows * cols)
                row = (idx[inside] - start) // cols
                vals = g[inside]
                vals[~active[row]] = 0.0
                g[inside] = vals
        return g

    def stored_gradient(self, worker: int, step: int, idx: Optional[np.ndarray] = None) -> np.ndarray:
        """The gradient as stored: fp32 values, or bf16 bit patterns (uint16)."""
        g = self.gradient(worker, step, idx)
        return hashgen.f32_to_bf16(g) if self.grad_dtype == "bf16" else g

    def subset(self, name: str, sizes, T: Optional[int] = None, K: Optional[int] = None,
               sparse="keep") -> "Workload":
        """Same rule and inputs on another tensor list (used for reduced-size cases)."""
        return Workload(name=name, K=self.K if K is None else K, sizes=tuple(int(s) for s in sizes),
                        T=self.T if T is None else T, lr=self.lr, momentum=self.momentum,
                        weight_decay=self.weight_decay, seed=self.seed, grad_kind=self.grad_kind,
                        grad_scale=self.grad_scale, grad_dtype=self.grad_dtype,
                        staleness=self.staleness,
                        sparse=self.sparse if sparse == "keep" else sparse, note=self.note)


def _load_sizes(name: str) -> Tuple[int, ...]:
    with open(os.path.join(_HERE, "layouts", name + ".json")) as f:
        return tuple(json.load(f)["sizes"])


def gru_sizes() -> Tuple[int, ...]:
    """Embedding 30k x 1024, 3-layer GRU (hidden 1024, input 512), projection 1024 -> 30k."""
    hid, inp, vocab = 1024, 512, 30_000
    sizes = [vocab * hid]
    for layer in range(3):
        in_dim = inp if layer == 0 else hid
        sizes += [3 * hid * in_dim, 3 * hid * hid, 3 * hid, 3 * hid]
    sizes += [vocab * hid, vocab]
    return tuple(sizes)


def make_workloads():
    w = {}
    w["cfg1"] = Workload("cfg1", K=4, sizes=(1_048_576,), T=10, lr=0.01, momentum=0.0,
                         weight_decay=0.0, seed=1, grad_kind="uniform", grad_scale=1e-2,
                         note="single flat tensor, plain SGD")
    w["cfg2"] = Workload("cfg2", K=8, sizes=_load_sizes("cfg2"), T=50, lr=0.1, momentum=0.9,
                         weight_decay=0.0, seed=2, grad_kind="gauss", grad_scale=1e-3,
                         note="ResNet-18-like: 62 tensors, 11.7M parameters")
    w["cfg3"] = Workload("cfg3", K=8, sizes=_load_sizes("cfg3"), T=50, lr=0.1, momentum=0.9,
                         weight_decay=5e-4, seed=3, grad_kind="gauss", grad_scale=1e-3,
                         note="ResNet-50-like: 161 tensors, 25.6M parameters, weight decay")
    w["cfg4"] = Workload("cfg4", K=16, sizes=_load_sizes("cfg4"), T=20, lr=0.01, momentum=0.9,
                         weight_decay=0.0, seed=4, grad_kind="gauss", grad_scale=1e-4,
                         note="VGG-16-like: 32 tensors, 138M parameters, FC-heavy")
    w["cfg5"] = Workload("cfg5", K=16, sizes=gru_sizes(), T=30, lr=0.01, momentum=0.9,
                         weight_decay=0.0, seed=5, grad_kind="gauss", grad_scale=1e-3,
                         grad_dtype="bf16", sparse=(0, 30_000, 1024),
                         note="GRU-shaped: bf16 gradients, sparse-row embedding gradient")
    return w


WORKLOADS = None


def get(name: str) -> Workload:
    global WORKLOADS
    if WORKLOADS is None:
        WORKLOADS = make_workloads()
    return WORKLOADS[name]


def names() -> List[str]:
    return ["cfg1", "cfg2", "cfg3", "cfg4", "cfg5"]
