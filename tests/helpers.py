"""Shared test helpers: building packed inputs from probability tables, reading
the hand-worked fixture, and classifying GPU-vs-oracle differences."""
from __future__ import annotations

import os

import numpy as np

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")
ZERO_LOGIT = np.float32(-1e30)   # stands for probability 0; exp() of it underflows to exactly 0


def probs_to_logits(rows) -> np.ndarray:
    """ln(prob) as float32, with probability 0 mapped to a very negative finite logit."""
    a = np.asarray(rows, dtype=np.float64)
    out = np.full(a.shape, ZERO_LOGIT, dtype=np.float32)
    np.log(a, where=a > 0, out=out, casting="unsafe")
    return out


def f32_to_bf16_bits(a: np.ndarray) -> np.ndarray:
    """Round float32 to bf16 (nearest even), returned as uint16 bit patterns."""
    bits = np.ascontiguousarray(a, dtype=np.float32).view(np.uint32).astype(np.uint64)
    rounded = (bits + 0x7FFF + ((bits >> 16) & 1)) >> 16
    return rounded.astype(np.uint16)


def bf16_bits_to_f64(a: np.ndarray) -> np.ndarray:
    return (a.astype(np.uint32) << 16).view(np.float32).astype(np.float64)


def logits_as_f64(a: np.ndarray) -> np.ndarray:
    return bf16_bits_to_f64(a) if a.dtype == np.uint16 else a.astype(np.float64)


def pack(seqs, V, dtype=np.float32):
    """Pack a list of sequences into the ragged layout.

    Each sequence is a dict with target (K+1, V) logits, draft (K, V) logits,
    tokens (K,), u (K,), u2 scalar.  Returns the six call arguments plus offsets.
    """
    B = len(seqs)
    k = np.array([len(s["tokens"]) for s in seqs], np.int32)
    D = int(k.sum())
    tl = np.zeros((D + B, V), dtype)
    dl = np.zeros((D, V), dtype)
    tok = np.zeros(D, np.int32)
    uni = np.zeros(D + B, np.float32)
    off_d = np.concatenate([[0], np.cumsum(k)]).astype(np.int64)
    off_t = off_d[:-1] + np.arange(B)
    for b, s in enumerate(seqs):
        K = int(k[b])
        tl[off_t[b]:off_t[b] + K + 1] = np.asarray(s["target"], dtype).reshape(K + 1, V)
        if K:
            dl[off_d[b]:off_d[b] + K] = np.asarray(s["draft"], dtype).reshape(K, V)
            tok[off_d[b]:off_d[b] + K] = s["tokens"]
            uni[off_t[b]:off_t[b] + K] = s["u"]
        uni[off_t[b] + K] = s["u2"]
    return tl, dl, tok, k, uni, off_d, off_t


def read_hand_cases():
    cases, cur = [], None
    with open(os.path.join(GOLDEN, "hand_cases.txt")) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            key, _, rest = line.partition(" ")
            if key == "case":
                cur = {"name": rest.strip(), "zero_margin": False, "no_crossing": False}
                cases.append(cur)
            elif key in ("target", "draft"):
                rows = [r.split() for r in rest.split(";")] if rest.strip() else []
                cur[key] = [[float(v) for v in r] for r in rows if r]
            elif key == "T":
                cur["T"] = float(rest)
            elif key == "tokens":
                cur["tokens"] = [int(v) for v in rest.split()]
            elif key in ("u", "expect_ptok", "expect_qtok", "expect_rho"):
                cur[key] = [float(v) for v in rest.split()]
            elif key == "expect_len":
                cur["expect_len"] = int(rest)
            elif key == "expect_emitted":
                cur["expect_emitted"] = [int(v) for v in rest.split()]
            elif key == "zero_margin":
                cur["zero_margin"] = True
            elif key == "no_crossing":
                cur["no_crossing"] = True
            else:
                raise ValueError(f"unknown key {key!r} in hand_cases.txt")
    return cases


def hand_case_inputs(case):
    """Packed call arguments (B=1) of one hand-worked case."""
    V = len(case["target"][0])
    K = len(case["tokens"])
    seq = {"target": probs_to_logits(case["target"]),
           "draft": probs_to_logits(case["draft"]) if K else np.zeros((0, V), np.float32),
           "tokens": case["tokens"], "u": case["u"][:K], "u2": case["u"][K]}
    tl, dl, tok, k, uni, _, _ = pack([seq], V)
    return tl, dl, tok, k, np.array([case["T"]], np.float32), uni


MARGIN = 1e-5


def classify_rows(ora, k_per_row, got_len, got_emitted, off_d, off_t, margin=MARGIN):
    """Compare accepted lengths and emitted tokens sequence by sequence.

    A sequence whose outputs differ is excused iff the oracle's own deciding
    margin is below `margin`: |u_i - rho_i| for some position i <= n_b (an accept
    decision that could flip), or the margin of the resample/bonus draw.
    Returns (identical, excused, failures) with failures a list of sequence ids.
    """
    identical, excused, failures = 0, 0, []
    B = len(k_per_row)
    for b in range(B):
        K = int(k_per_row[b])
        sl = slice(int(off_t[b]), int(off_t[b]) + K + 1)
        same = (int(got_len[b]) == int(ora.accepted_len[b])
                and np.array_equal(np.asarray(got_emitted[sl]), ora.emitted_tokens[sl]))
        if same:
            identical += 1
            continue
        n = int(ora.accepted_len[b])
        am = ora.accept_margin[int(off_d[b]):int(off_d[b]) + min(n + 1, K)]
        thin_accept = am.size > 0 and float(np.nanmin(am)) < margin
        thin_cdf = bool(ora.cdf_margin[b] < margin)
        if thin_accept or thin_cdf:
            excused += 1
        else:
            failures.append(b)
    return identical, excused, failures


class Case:
    """Packed numpy arrays with the Workload fields the test helpers use."""
    def __init__(self, tl, dl, tok, k, T, uni, dtype="f32"):
        self.target_logits, self.draft_logits, self.draft_tokens = tl, dl, tok
        self.k_per_row, self.temperature, self.uniforms = k, T, uni
        self.B, self.V, self.dtype = len(k), tl.shape[1], dtype
        self.off_d = np.concatenate([[0], np.cumsum(k)]).astype(np.int64)
        self.off_t = self.off_d[:-1] + np.arange(self.B)
        self.n_draft_total = int(self.off_d[-1])


def neg_inf_of(a: np.ndarray):
    """-inf in the storage type of a logits array (bf16 is stored as uint16 bit patterns)."""
    return np.uint16(0xFF80) if a.dtype == np.uint16 else a.dtype.type(-np.inf)


def masked_case(w, seed: int, contiguous_every: int = 3):
    """Workload w with half of every sequence's vocabulary masked by -inf logits, the way a
    constrained sampler masks forbidden tokens: per sequence one set of kept ids (exactly
    V // 2 of them), applied to all its target and draft rows; every `contiguous_every`-th
    sequence keeps the SECOND half of the vocabulary instead of a random half, so that whole
    vectors, lanes and chunks of a row hold nothing but -inf.  Drafted tokens are moved onto
    kept ids.  Returns (case, kept) with kept[b] the sorted kept ids of sequence b."""
    rng = np.random.default_rng(seed)
    tl, dl, tok = w.target_logits.copy(), w.draft_logits.copy(), w.draft_tokens.copy()
    ninf = neg_inf_of(tl)
    V, kept = w.V, []
    for b in range(w.B):
        if b % contiguous_every == contiguous_every - 1:
            keep = np.arange(V - V // 2, V)
        else:
            keep = np.sort(rng.choice(V, V // 2, replace=False))
        kept.append(keep)
        gone = np.ones(V, bool)
        gone[keep] = False
        K = int(w.k_per_row[b])
        tl[w.off_t[b]:w.off_t[b] + K + 1, gone] = ninf
        dl[w.off_d[b]:w.off_d[b] + K, gone] = ninf
        for i in range(K):
            x = tok[w.off_d[b] + i]
            tok[w.off_d[b] + i] = keep[np.searchsorted(keep, x) % len(keep)]
    return Case(tl, dl, tok, w.k_per_row, w.temperature, w.uniforms, dtype=w.dtype), kept
