"""Fragment tables and hyper-parameters of the synthetic workloads.

Every workload is a flat vector of N fp32 parameters cut into K disjoint
fragments (the paper partitions the model along its depth, Section 2.1).  A
fragment is a list of contiguous segments; most fragments have one, the
"embeddings" fragments of the transformer-shaped workloads have two (the
token table at the front of the vector, the final norm / output head at its
end), which is also how a strided shard looks (Section 4.1).

Shapes are public architecture arithmetic only (layer counts and widths);
no trained weights, datasets or benchmark items are involved.
"""

from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import List, Sequence, Tuple

import numpy as np

Segment = Tuple[int, int]  # (element offset into every N-sized buffer, length)


@dataclass(frozen=True)
class Partition:
    """K fragments over a flat vector of N elements, CSR over segments."""

    N: int
    fragments: Tuple[Tuple[Segment, ...], ...]

    @property
    def K(self) -> int:
        return len(self.fragments)

    @property
    def n_segments(self) -> int:
        return sum(len(f) for f in self.fragments)

    def frag_size(self, p: int) -> int:
        return sum(l for _, l in self.fragments[p])

    @property
    def frag_sizes(self) -> np.ndarray:
        return np.array([self.frag_size(p) for p in range(self.K)], dtype=np.int64)

    def csr(self):
        """(frag_seg_ptr int32[K+1], seg_offset int64[S], seg_len int64[S])."""
        ptr = [0]
        off: List[int] = []
        ln: List[int] = []
        for f in self.fragments:
            for o, l in f:
                off.append(o)
                ln.append(l)
            ptr.append(len(off))
        return (np.asarray(ptr, dtype=np.int32), np.asarray(off, dtype=np.int64),
                np.asarray(ln, dtype=np.int64))

    def check(self) -> None:
        segs = sorted((o, l) for f in self.fragments for o, l in f)
        end = 0
        for o, l in segs:
            assert l > 0 and o >= end and o + l <= self.N, (o, l, end, self.N)
            end = o + l


def contiguous_partition(sizes: Sequence[int]) -> Partition:
    frags = []
    off = 0
    for s in sizes:
        frags.append(((off, int(s)),))
        off += int(s)
    return Partition(N=off, fragments=tuple(frags))


@dataclass(frozen=True)
class Workload:
    name: str
    partition: Partition
    M: int                      # worker replicas
    tau: int                    # overlap depth (delay in local steps)
    H: int = 100                # local steps between syncs of a fragment (Section 4.1)
    outer_lr: float = 0.7
    momentum: float = 0.9
    lam: float = 0.5            # compensation strength lambda
    alpha: float = 1.0          # mixing factor; 1 = assignment of the corrected target
    budget_kind: str = "count"  # "count" (fragments) or "params" (elements)
    budget: int = 1
    seed: int = 0
    scale_kind: str = "const"   # per-fragment drift scale: const | loguniform | student_t
    sigma_global: float = 0.02  # global parameters ~ N(0, sigma_global)
    sigma_drift: float = 1e-3   # worker drift and change over the delay ~ N(0, sigma_drift)
    notes: str = ""

    @property
    def N(self) -> int:
        return self.partition.N

    @property
    def K(self) -> int:
        return self.partition.K

    def with_(self, **kw) -> "Workload":
        return replace(self, **kw)


# --------------------------------------------------------------------------
# the five workloads
# --------------------------------------------------------------------------

def _tiny() -> Workload:
    return Workload(
        name="tiny", partition=contiguous_partition([131072] * 8), M=2, tau=1,
        outer_lr=0.7, momentum=0.9, lam=0.5, budget_kind="count", budget=2, seed=0,
        scale_kind="const", notes="1,048,576 params, 8 equal fragments")


def _gpt2_small() -> Workload:
    d, layers, vocab, ctx = 768, 12, 50257, 1024
    layer = 12 * d * d + 13 * d                 # attention + MLP + two norms, with biases
    front = vocab * d + ctx * d                 # token + position tables
    tail = 2 * d                                # final norm
    N = front + layers * layer + tail
    frags = [((0, front), (N - tail, tail))]    # embeddings fragment: two segments
    for i in range(layers):
        frags.append(((front + i * layer, layer),))
    part = Partition(N=N, fragments=tuple(frags))
    return Workload(
        name="gpt2_small", partition=part, M=4, tau=2, budget_kind="params",
        budget=N // 4, seed=1, scale_kind="loguniform",
        notes="GPT-2-small-shaped: 12 layers d=768 + embeddings, 13 ragged fragments")


def _llama_shape(layers: int, d: int, ffn: int, vocab: int):
    layer = 4 * d * d + 3 * d * ffn + 2 * d
    embed = vocab * d
    return layer, embed, d  # final norm has d elements


def _llama_1b() -> Workload:
    layers = 16
    layer, embed, norm = _llama_shape(layers, 2048, 5632, 32000)
    sizes = [embed + layer] + [layer] * (layers - 2) + [layer + norm + embed]
    return Workload(
        name="llama_1b", partition=contiguous_partition(sizes), M=4, tau=4,
        budget_kind="count", budget=4, seed=2, scale_kind="loguniform",
        notes="Llama-1B-shaped: 16 layer-aligned fragments")


def _sweep_1b() -> Workload:
    layers = 16
    layer, embed, norm = _llama_shape(layers, 2048, 5632, 32000)
    N = 2 * embed + layers * layer + norm
    assert N % 32 == 0
    return Workload(
        name="sweep_1b", partition=contiguous_partition([N // 32] * 32), M=4, tau=4,
        budget_kind="count", budget=32, seed=3, scale_kind="const",
        notes="1B shape cut into 32 equal fragments (compensation sweep)")


def _llama_3b() -> Workload:
    layers = 26
    layer, embed, norm = _llama_shape(layers, 3200, 8640, 32000)
    N = 2 * embed + layers * layer + norm
    frags = []
    for i in range(layers):
        frags.append(((embed + i * layer, layer),))
    # embeddings fragment: token table at the front, final norm + output head at the end
    frags.append(((0, embed), (embed + layers * layer, norm + embed)))
    part = Partition(N=N, fragments=tuple(frags))
    return Workload(
        name="llama_3b", partition=part, M=4, tau=4, budget_kind="params",
        budget=(3 * N) // 10, seed=4, scale_kind="student_t",
        notes="Llama-3B-shaped: 26 layer fragments + one embeddings fragment")


def _paper_150m() -> Workload:
    """The shape of the paper's own experiment (Section 4.1): a LLaMA-style decoder of 12 layers and about
    150 M parameters cut into 4 shards of 3 layers in a strided pattern, M = 4, H = 100, tau = 5, lambda = 0.5,
    one fragment per decision (Algorithm 2).  Width 1024 / FFN 2816 give 12.85 M parameters per layer."""
    layers, shards = 12, 4
    layer, _, _ = _llama_shape(layers, 1024, 2816, 32000)
    frags = [tuple((l * layer, layer) for l in range(k, layers, shards)) for k in range(shards)]
    part = Partition(N=layers * layer, fragments=tuple(frags))
    return Workload(
        name="paper_150m", partition=part, M=4, tau=5, H=100, lam=0.5, budget_kind="count", budget=1, seed=5,
        scale_kind="loguniform", notes="12 layers in 4 strided shards of 3 layers (Section 4.1)")


_BUILDERS = {
    "tiny": _tiny,
    "gpt2_small": _gpt2_small,
    "llama_1b": _llama_1b,
    "sweep_1b": _sweep_1b,
    "llama_3b": _llama_3b,
    "paper_150m": _paper_150m,
}
WORKLOAD_NAMES = tuple(_BUILDERS)


def get_workload(name: str) -> Workload:
    w = _BUILDERS[name]()
    w.partition.check()
    return w


def small_workload(sizes_or_fragments, M: int, seed: int = 0, **kw) -> Workload:
    """A test-sized workload.

    `sizes_or_fragments` is either a list of fragment sizes (laid out back to
    back) or a (N, list of fragments, each a list of (offset, len)) pair for
    gaps, odd offsets and strided fragments.
    """
    if isinstance(sizes_or_fragments, tuple) and len(sizes_or_fragments) == 2 \
            and not isinstance(sizes_or_fragments[0], (tuple, list)):
        N, frs = sizes_or_fragments
        part = Partition(N=int(N), fragments=tuple(tuple((int(o), int(l)) for o, l in f) for f in frs))
    else:
        part = contiguous_partition(list(sizes_or_fragments))
    part.check()
    kw.setdefault("tau", 2)
    return Workload(name=kw.pop("name", "small"), partition=part, M=M, seed=seed, **kw)
