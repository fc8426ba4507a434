"""Seeded synthetic inputs for the verify-and-resample pass.

This module only manufactures inputs (logits, drafted tokens, uniforms, lookahead
lengths, temperatures) in the packed ragged layout; it contains none of the method's
arithmetic -- no softmax, no acceptance test, no cumulative sums.  Drafted tokens are
drawn from softmax(draft_logits / T) with the Gumbel-max trick (argmax of tempered
logit plus Gumbel noise), which needs no probabilities.

The five workloads stand in for real language-model logits: vocabulary sizes 32000,
128256 and 152064 are those of common open tokenizers, the Zipf-shaped rows mimic the
heavy-tailed next-token distributions of trained models, and the ragged lookahead of
the last workload is the paper's input-dependent speculation (section "Dynamic
Execution": the amount of speculative work depends on the input).

Every row has its own counter-based stream (Philox keyed by seed and row), so a
workload is the same bytes however many threads generate it.
"""
from __future__ import annotations

import os
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass, field

import numpy as np


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16, nearest-even, as uint16 bit patterns (finite inputs)."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32)
    rounded = (bits + (np.uint32(0x7FFF) + ((bits >> np.uint32(16)) & np.uint32(1)))) >> np.uint32(16)
    return rounded.astype(np.uint16)


def bf16_bits_to_f32(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << np.uint32(16)).view(np.float32)


@dataclass
class Workload:
    name: str
    B: int
    V: int
    dtype: str                    # "f32", "f16" or "bf16" (bf16 stored as uint16 bit patterns)
    k_per_row: np.ndarray         # int32 [B]
    target_logits: np.ndarray     # [sum(K)+B, V]
    draft_logits: np.ndarray      # [sum(K), V]
    draft_tokens: np.ndarray      # int32 [sum(K)]
    temperature: np.ndarray       # float32 [1] or [B]
    uniforms: np.ndarray          # float32 [sum(K)+B]
    off_d: np.ndarray = field(default=None)   # int64 [B+1]
    off_t: np.ndarray = field(default=None)   # int64 [B]
    recipe: str = ""

    @property
    def n_draft_total(self) -> int:
        return int(self.off_d[-1])

    @property
    def logit_bytes(self) -> int:
        """Bytes of logits, every row once: the algorithmic traffic of one verify pass."""
        elt = 4 if self.dtype == "f32" else 2
        return (2 * self.n_draft_total + self.B) * self.V * elt

    def take(self, b0: int, b1: int) -> "Workload":
        """The sub-batch of sequences b0..b1-1 (views, nothing regenerated)."""
        d0, d1 = int(self.off_d[b0]), int(self.off_d[b1])
        t0, t1 = d0 + b0, d1 + b1
        temp = self.temperature if self.temperature.shape[0] == 1 else self.temperature[b0:b1]
        k = self.k_per_row[b0:b1]
        off_d = np.concatenate([[0], np.cumsum(k)]).astype(np.int64)
        return Workload(f"{self.name}[{b0}:{b1}]", b1 - b0, self.V, self.dtype, k,
                        self.target_logits[t0:t1], self.draft_logits[d0:d1],
                        self.draft_tokens[d0:d1], temp, self.uniforms[t0:t1],
                        off_d, off_d[:-1] + np.arange(b1 - b0), self.recipe)


# name -> (B, K spec, V, dtype, seed)
_SPECS = {
    1: dict(B=1, K=4, V=32000, dtype="f32", seed=0,
            recipe="target N(0,3^2) iid; draft = target + N(0,1); T=1.0"),
    2: dict(B=8, K=5, V=32000, dtype="bf16", seed=1,
            recipe="target N(0,3^2); draft = 0.9*target + N(0,1.5^2); T=0.7"),
    3: dict(B=64, K=8, V=128256, dtype="bf16", seed=2,
            recipe="target Zipf-shaped: sorted N(0,1) + 8*(rank+1)^-0.5, permuted per row; "
                   "draft = target + N(0,1); T=1.0"),
    4: dict(B=256, K=4, V=152064, dtype="bf16", seed=3,
            recipe="target N(0,4^2); draft = target + N(0,0.5^2); per-sequence T ~ U[0.3,1.2]"),
    5: dict(B=512, K="ragged 1..16", V=128256, dtype="bf16", seed=4,
            recipe="ragged K_b ~ U{1..16}; target N(0,3^2); draft = target + N(0,s_b^2), "
                   "s_b ~ U[0.3,2.0] per sequence; T=0.8"),
}

_STREAM_ROWS, _STREAM_SCALARS, _STREAM_UNIFORMS = 0, 1, 2


def _rng(seed: int, stream: int, index: int) -> np.random.Generator:
    return np.random.Generator(np.random.Philox(key=[(seed << 8) | stream, index]))


def _target_row(cfg: int, g: np.random.Generator, V: int) -> np.ndarray:
    z = g.standard_normal(V, dtype=np.float32)
    if cfg in (1, 2, 5):
        return z * np.float32(3.0)
    if cfg == 4:
        return z * np.float32(4.0)
    # cfg 3: heavy-tailed row -- largest normal gets the largest boost, then shuffle
    z = -np.sort(-z)
    z += (np.float32(8.0) * (np.arange(1, V + 1, dtype=np.float64) ** -0.5)).astype(np.float32)
    return z[g.permutation(V)]


def make_config(cfg: int, *, B: int | None = None, V: int | None = None, K: int | None = None,
                threads: int | None = None, dtype: str | None = None) -> Workload:
    """Workload `cfg` (1..5).  B, V, K override the size (same recipe, same seed) for
    small parity cases; K overrides only the fixed-K workloads; dtype ("f32", "bf16", "f16")
    overrides the storage type of the logits."""
    spec = dict(_SPECS[cfg])
    if dtype is not None:
        spec["dtype"] = dtype
    B = spec["B"] if B is None else B
    V = spec["V"] if V is None else V
    seed = spec["seed"]
    gs = _rng(seed, _STREAM_SCALARS, 0)
    if cfg == 5:
        k = gs.integers(1, 17, size=B).astype(np.int32)
    else:
        k = np.full(B, spec["K"] if K is None else K, np.int32)
    if cfg == 4:
        temperature = gs.uniform(0.3, 1.2, size=B).astype(np.float32)
    else:
        temperature = np.array([{1: 1.0, 2: 0.7, 3: 1.0, 5: 0.8}[cfg]], np.float32)
    sigma = gs.uniform(0.3, 2.0, size=B).astype(np.float32) if cfg == 5 else None

    off_d = np.concatenate([[0], np.cumsum(k)]).astype(np.int64)
    off_t = off_d[:-1] + np.arange(B)
    D = int(off_d[-1])
    store = {"f32": np.float32, "bf16": np.uint16, "f16": np.float16}[spec["dtype"]]
    tl = np.empty((D + B, V), store)
    dl = np.empty((D, V), store)
    tok = np.empty(D, np.int32)

    def to_store(a):
        if store is np.float32:
            return a
        return f32_to_bf16_bits(a) if store is np.uint16 else a.astype(np.float16)

    def as_f32(a):
        if store is np.float32:
            return a
        return bf16_bits_to_f32(a) if store is np.uint16 else a.astype(np.float32)

    def fill(b: int):
        T = float(temperature[b] if temperature.shape[0] > 1 else temperature[0])
        for i in range(int(k[b]) + 1):
            g = _rng(seed, _STREAM_ROWS, (b << 8) | i)
            t = _target_row(cfg, g, V)
            tl[off_t[b] + i] = to_store(t)
            if i == int(k[b]):
                break
            noise = g.standard_normal(V, dtype=np.float32)
            if cfg == 1:
                d = t + noise
            elif cfg == 2:
                d = np.float32(0.9) * t + np.float32(1.5) * noise
            elif cfg == 3:
                d = t + noise
            elif cfg == 4:
                d = t + np.float32(0.5) * noise
            else:
                d = t + sigma[b] * noise
            ds = to_store(d)
            dl[off_d[b] + i] = ds
            # Gumbel-max draw from softmax(draft / T): argmax(logit/T - ln(Exp(1) sample))
            e = g.standard_exponential(V, dtype=np.float32)
            np.maximum(e, np.float32(1e-38), out=e)
            tok[off_d[b] + i] = int(np.argmax(as_f32(ds) / np.float32(T) - np.log(e)))

    threads = threads or min(32, os.cpu_count() or 1)
    if threads > 1 and B > 1:
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(fill, range(B)))
    else:
        for b in range(B):
            fill(b)

    gu = _rng(seed, _STREAM_UNIFORMS, 0)
    uniforms = (gu.integers(0, 1 << 24, size=D + B).astype(np.float32) * np.float32(2.0 ** -24))
    return Workload(f"config{cfg}", B, V, spec["dtype"], k, tl, dl, tok, temperature, uniforms,
                    off_d, off_t, spec["recipe"])


def describe(cfg: int) -> str:
    s = _SPECS[cfg]
    return f"B={s['B']} K={s['K']} V={s['V']} {s['dtype']} seed={s['seed']}: {s['recipe']}"


# ----------------------------------------------------------------------------- draft trees
@dataclass
class TreeWorkload(Workload):
    """A Workload whose drafts form a tree per sequence: k_per_row holds the node counts N_b,
    draft_tokens the node tokens, node_parent the parent of every node (-1 = root).  Target row c
    of a sequence belongs to context c (0 = root, j+1 = after node j); draft row c is the
    distribution the children of context c were drawn from, and is filled with NaN when the
    context has none (such rows must never be read)."""
    node_parent: np.ndarray = field(default=None)     # int32 [sum(N)]
    n_internal: int = 0                               # contexts that have children, whole batch

    @property
    def logit_bytes(self) -> int:
        """Every target row and every draft row of a context with children, once."""
        elt = 4 if self.dtype == "f32" else 2
        return (self.n_draft_total + self.B + self.n_internal) * self.V * elt

    def take(self, b0: int, b1: int) -> "TreeWorkload":
        base = Workload.take(self, b0, b1)
        d0, d1 = int(self.off_d[b0]), int(self.off_d[b1])
        par = self.node_parent[d0:d1]
        internal = 0
        for b in range(b0, b1):
            p = self.node_parent[int(self.off_d[b]):int(self.off_d[b + 1])]
            internal += len(set(int(x) for x in p))
        return TreeWorkload(base.name, base.B, base.V, base.dtype, base.k_per_row, base.target_logits,
                            base.draft_logits, base.draft_tokens, base.temperature, base.uniforms,
                            base.off_d, base.off_t, base.recipe, node_parent=par, n_internal=internal)


def make_tree_config(*, B: int = 64, V: int = 128256, dtype: str = "bf16", seed: int = 5,
                     max_level_width: int = 6, depth: int = 5, temperature: float = 0.8,
                     threads: int | None = None) -> TreeWorkload:
    """Seeded batch of draft trees, shaped like the candidate trees of tree-drafting methods:
    `depth` levels below the root, level widths drawn per sequence from 1..max_level_width
    (non-increasing), every node attached to a parent of the level above with a preference for the
    first (most probable) ones.  Nodes are numbered level by level, so a parent precedes its
    children.  Logits as in workload 5: target N(0,3^2), draft = target + N(0,s_b^2) with
    s_b ~ U[0.3,2.0] per sequence; the children of a context are independent Gumbel-max draws from
    softmax(draft row / T)."""
    gs = _rng(seed, _STREAM_SCALARS, 0)
    parents, counts = [], []
    for b in range(B):
        widths, wmax = [], max_level_width
        for _ in range(depth):
            wl = int(gs.integers(1, wmax + 1))
            widths.append(wl)
            wmax = wl
        par, level_nodes = [], [-1]                 # the root stands for the level above level 0
        for wl in widths:
            first = len(par)
            for _ in range(wl):
                # geometric preference for the first parents of the level above
                pick = min(int(gs.geometric(0.55)) - 1, len(level_nodes) - 1)
                par.append(level_nodes[pick])
            order = np.argsort(par[first:], kind="stable")      # children of one parent stay together
            par[first:] = [par[first + i] for i in order]
            level_nodes = list(range(first, first + wl))
        parents.append(np.array(par, np.int32))
        counts.append(len(par))
    n = np.array(counts, np.int32)
    sigma = gs.uniform(0.3, 2.0, size=B).astype(np.float32)
    T = np.array([temperature], np.float32)
    off_d = np.concatenate([[0], np.cumsum(n)]).astype(np.int64)
    off_t = off_d[:-1] + np.arange(B)
    D = int(off_d[-1])
    store = {"f32": np.float32, "bf16": np.uint16, "f16": np.float16}[dtype]
    tl = np.empty((D + B, V), store)
    dl = np.empty((D, V), store)
    if store is np.uint16:
        dl[:] = 0x7FC0                              # bf16 NaN
    else:
        dl[:] = np.nan
    tok = np.empty(D, np.int32)
    internal = [0] * B

    def to_store(a):
        if store is np.float32:
            return a
        return f32_to_bf16_bits(a) if store is np.uint16 else a.astype(np.float16)

    def as_f32(a):
        if store is np.float32:
            return a
        return bf16_bits_to_f32(a) if store is np.uint16 else a.astype(np.float32)

    def fill(b: int):
        par = parents[b]
        N = int(n[b])
        for c in range(N + 1):
            g = _rng(seed, _STREAM_ROWS, (b << 8) | c)
            t = g.standard_normal(V, dtype=np.float32) * np.float32(3.0)
            tl[off_t[b] + c] = to_store(t)
            kids = np.nonzero(par == c - 1)[0]
            if kids.size == 0:
                continue
            internal[b] += 1
            ds = to_store(t + sigma[b] * g.standard_normal(V, dtype=np.float32))
            dl[off_d[b] + c] = ds
            scaled = as_f32(ds) / np.float32(temperature)
            for j in kids:                          # independent draws from softmax(draft / T)
                e = g.standard_exponential(V, dtype=np.float32)
                np.maximum(e, np.float32(1e-38), out=e)
                tok[off_d[b] + j] = int(np.argmax(scaled - np.log(e)))

    threads = threads or min(32, os.cpu_count() or 1)
    if threads > 1 and B > 1:
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(fill, range(B)))
    else:
        for b in range(B):
            fill(b)
    gu = _rng(seed, _STREAM_UNIFORMS, 0)
    uniforms = (gu.integers(0, 1 << 24, size=D + B).astype(np.float32) * np.float32(2.0 ** -24))
    recipe = (f"draft trees: {depth} levels of 1..{max_level_width} nodes (non-increasing), children are "
              f"independent draws from the draft row; target N(0,3^2); draft = target + N(0,s_b^2), "
              f"s_b ~ U[0.3,2.0]; T={temperature}")
    return TreeWorkload("tree", B, V, dtype, n, tl, dl, tok, T, uniforms, off_d, off_t, recipe,
                        node_parent=np.concatenate(parents).astype(np.int32), n_internal=int(sum(internal)))


# ----------------------------------------------------------------------------- hidden states
@dataclass
class HiddenWorkload:
    """Inputs of the verify pass one step earlier: hidden states and output-layer weights of both
    models (bf16 bit patterns), from which the logits are a matrix product.  The draft tokens must be
    drawn from the draft logits, which this module does not compute (no arithmetic of the method
    here): the caller computes them with its own LM-head product and calls draw_tokens()."""
    B: int
    V: int
    k_per_row: np.ndarray
    target_hidden: np.ndarray     # uint16 [sum(K)+B, H]
    target_weight: np.ndarray     # uint16 [V, H]
    draft_hidden: np.ndarray      # uint16 [sum(K), Hd]
    draft_weight: np.ndarray      # uint16 [V, Hd]
    temperature: np.ndarray
    uniforms: np.ndarray
    off_d: np.ndarray
    off_t: np.ndarray
    seed: int

    @property
    def n_draft_total(self) -> int:
        return int(self.off_d[-1])

    def draw_tokens(self, draft_logits_bits: np.ndarray) -> np.ndarray:
        """Draft tokens by Gumbel-max from softmax(draft logits / T) (bf16 bit patterns in)."""
        tok = np.empty(self.n_draft_total, np.int32)
        for b in range(self.B):
            T = float(self.temperature[b] if self.temperature.shape[0] > 1 else self.temperature[0])
            for i in range(int(self.k_per_row[b])):
                g = _rng(self.seed, _STREAM_ROWS, (b << 8) | i)
                e = g.standard_exponential(self.V, dtype=np.float32)
                np.maximum(e, np.float32(1e-38), out=e)
                row = bf16_bits_to_f32(draft_logits_bits[self.off_d[b] + i])
                tok[self.off_d[b] + i] = int(np.argmax(row / np.float32(T) - np.log(e)))
        return tok


def make_hidden_config(*, B: int, V: int, H: int, Hd: int | None = None, K: int | None = None, seed: int = 6,
                       exact: bool = True, temperature: float = 0.8) -> HiddenWorkload:
    """Seeded hidden states and weights.  exact=True: every product and every sum of the matrix
    product is exactly representable -- hidden states with 24 non-zero entries per row from
    {+-1/4, +-1/2}, weights integers in [-2, 2] -- so the logits are multiples of 1/4 below 32 in
    magnitude, which bf16 holds exactly, and any correct product gives the same bytes whatever its
    accumulation order.  The draft model's hidden state is the target's with a third of the non-zero
    entries redrawn (so the two models mostly agree); exact=False: N(0,1) hidden states and
    N(0, 1/H) weights (no exactness; for timing).  K: fixed lookahead, else ragged 1..8."""
    Hd = H if Hd is None else Hd
    g = _rng(seed, _STREAM_SCALARS, 0)
    k = np.full(B, K, np.int32) if K is not None else g.integers(1, 9, size=B).astype(np.int32)
    off_d = np.concatenate([[0], np.cumsum(k)]).astype(np.int64)
    off_t = off_d[:-1] + np.arange(B)
    D = int(off_d[-1])
    if exact:
        def sparse_rows(n, width, gen):
            a = np.zeros((n, width), np.float32)
            for r in range(n):
                idx = gen.choice(width, size=min(24, width), replace=False)
                a[r, idx] = gen.choice(np.array([-0.5, -0.25, 0.25, 0.5], np.float32), size=idx.size)
            return a
        th = sparse_rows(D + B, H, g)
        dh = np.zeros((D, Hd), np.float32)
        for b in range(B):
            for i in range(int(k[b])):
                row = th[off_t[b] + i, :min(H, Hd)].copy()
                nz = np.nonzero(row)[0]
                redo = nz[g.random(nz.size) < 1.0 / 3.0]
                row[redo] = g.choice(np.array([-0.5, -0.25, 0.25, 0.5], np.float32), size=redo.size)
                dh[off_d[b] + i, :row.size] = row
        tw = g.integers(-2, 3, size=(V, H)).astype(np.float32)
        dw = tw[:, :Hd].copy() if Hd <= H else np.concatenate([tw, g.integers(-2, 3, size=(V, Hd - H)).astype(np.float32)], 1)
    else:
        th = g.standard_normal((D + B, H), dtype=np.float32)
        dh = g.standard_normal((D, Hd), dtype=np.float32)
        tw = g.standard_normal((V, H), dtype=np.float32) * np.float32(3.0 / np.sqrt(H))
        dw = g.standard_normal((V, Hd), dtype=np.float32) * np.float32(3.0 / np.sqrt(Hd))
    gu = _rng(seed, _STREAM_UNIFORMS, 0)
    uniforms = gu.integers(0, 1 << 24, size=D + B).astype(np.float32) * np.float32(2.0 ** -24)
    return HiddenWorkload(B, V, k, f32_to_bf16_bits(th), f32_to_bf16_bits(tw), f32_to_bf16_bits(dh), f32_to_bf16_bits(dw),
                          np.array([temperature], np.float32), uniforms, off_d, off_t, seed)
