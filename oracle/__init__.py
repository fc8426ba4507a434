"""fp64 CPU oracle for the verify-and-resample pass (TEST INFRASTRUCTURE ONLY).

This package wraps ``spec_verify_oracle.c`` (plain C, double precision) with
ctypes.  It defines what the CUDA library must compute and is used by the tests,
by the smoke check and by the benchmark's CPU-baseline leg -- never by the
product path, and it imports nothing from the CUDA package.

The method it states is the one the paper's section "Speculative Sampling
Results" describes in prose: compare target and draft probabilities on the
drafted tokens, keep tokens up to the first rejection, resample the rejected
token from a combination of the two distributions, or sample one extra token
from the target when everything was accepted.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
from concurrent.futures import ThreadPoolExecutor
from dataclasses import dataclass

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "spec_verify_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_LIB_SAN = os.path.join(_HERE, "liboracle_san.so")
# ORACLE_SANITIZE=1: load the build instrumented with AddressSanitizer and
# UndefinedBehaviorSanitizer (the process must have libasan preloaded)
_SANITIZE = os.environ.get("ORACLE_SANITIZE", "") not in ("", "0")

F32 = 0
BF16 = 1
F16 = 2

ROW_BAD_K = 1
ROW_BAD_TEMPERATURE = 2
ROW_BAD_TOKEN = 4
ROW_ZERO_RESIDUAL = 8
ROW_BAD_PARENT = 32


def build(force: bool = False, sanitize: bool = False) -> str:
    """Compile the C oracle with gcc (no fast-math, no FMA contraction).  sanitize: the build
    with -fsanitize=address,undefined (same arithmetic flags)."""
    lib = _LIB_SAN if sanitize else _LIB
    stale = (not os.path.exists(lib)) or os.path.getmtime(lib) < os.path.getmtime(_SRC)
    if force or stale:
        tmp = lib + f".{os.getpid()}.tmp"
        extra = ["-fsanitize=address,undefined", "-fno-omit-frame-pointer", "-g"] if sanitize else []
        subprocess.check_call(
            ["gcc", "-std=c99", "-O2", "-ffp-contract=off", "-fno-fast-math", "-fPIC", "-shared", *extra,
             "-o", tmp, _SRC, "-lm"])
        os.replace(tmp, lib)
    return lib


_lib = None


def _load():
    global _lib
    if _lib is None:
        lib = ctypes.CDLL(build(sanitize=_SANITIZE))
        vp, i32, i64 = ctypes.c_void_p, ctypes.c_int32, ctypes.c_int64
        lib.oracle_spec_verify.restype = ctypes.c_int
        lib.oracle_spec_verify.argtypes = [
            vp, vp, ctypes.c_int, i64, i64, i64, vp, vp, i32, i32, i64, vp, ctypes.c_int, vp,
            i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_position_distributions.restype = ctypes.c_int
        lib.oracle_position_distributions.argtypes = [
            vp, vp, ctypes.c_int, i64, ctypes.c_double, vp, vp, vp]
        lib.oracle_next_lookahead.restype = None
        lib.oracle_next_lookahead.argtypes = [vp, i32, vp, i32, i32, i32, vp]
        lib.oracle_spec_verify_tree.restype = ctypes.c_int
        lib.oracle_spec_verify_tree.argtypes = [
            vp, vp, ctypes.c_int, i64, i64, i64, vp, vp, vp, i32, i32, i64, vp, ctypes.c_int, vp,
            i32, i32, vp, vp, vp, vp, vp, vp, vp, vp]
        lib.oracle_lm_head.restype = None
        lib.oracle_lm_head.argtypes = [vp, i64, vp, i64, i64, i64, i64, i64, i64, vp, i64]
        lib.oracle_spec_verify_greedy.restype = None
        lib.oracle_spec_verify_greedy.argtypes = [
            vp, ctypes.c_int, i64, i64, vp, vp, i32, i32, i64, i32, i32, vp, vp, vp, vp]
        _lib = lib
    return _lib


def _ptr(a):
    return None if a is None else a.ctypes.data_as(ctypes.c_void_p)


@dataclass
class OracleResult:
    accepted_len: np.ndarray      # int32 [B]
    emitted_tokens: np.ndarray    # int32 [n_draft_total + B], target packing, -1 padded
    row_status: np.ndarray        # int32 [B]
    p_tok: np.ndarray             # float64 [n_draft_total]  p_i(x_i)
    q_tok: np.ndarray             # float64 [n_draft_total]  q_i(x_i)
    rho: np.ndarray               # float64 [n_draft_total]  p_i(x_i) / q_i(x_i)
    accept_margin: np.ndarray     # float64 [n_draft_total]  |u_i - rho_i|
    cdf_margin: np.ndarray        # float64 [B]              margin of the resample / bonus draw


def _dtype_code(logits: np.ndarray) -> int:
    if logits.dtype == np.float32:
        return F32
    if logits.dtype == np.uint16:   # bf16 bit patterns
        return BF16
    if logits.dtype == np.float16:
        return F16
    raise TypeError("logits must be float32, float16 or uint16 (bf16 bit patterns)")


def spec_verify(target_logits, draft_logits, draft_tokens, k_per_row, temperature, uniforms,
                *, k_uniform: int = 0, threads: int = 1, b_range=None) -> OracleResult:
    """Run the oracle on host arrays.

    target_logits  [n_draft_total + B, ld_target] float32, or uint16 holding bf16 bits
    draft_logits   [n_draft_total, ld_draft]      same dtype
    draft_tokens   int32 [n_draft_total]
    k_per_row      int32 [B], or an int B when every sequence has k_uniform drafts
    temperature    float32 [1] or [B]
    uniforms       float32 [n_draft_total + B]
    threads        sequences are dealt to this many threads (the C call drops the GIL)
    b_range        (begin, end): only these sequences are computed; other outputs stay -1 / NaN
    The vocabulary size V is the logits' last dimension; a padded leading
    dimension is expressed by passing a sliced view ``a[:, :V]`` of a wider array.
    """
    lib = _load()
    tl, dl = target_logits, draft_logits
    dtype = _dtype_code(tl)
    assert dl.dtype == tl.dtype
    V = tl.shape[1]
    elt = tl.dtype.itemsize
    assert tl.strides[1] == elt and (dl.size == 0 or dl.strides[1] == elt)
    ld_t = tl.strides[0] // elt
    ld_d = dl.strides[0] // elt if dl.shape[0] > 0 else V
    if isinstance(k_per_row, (int, np.integer)):
        B, kpr = int(k_per_row), None
    else:
        kpr = np.ascontiguousarray(k_per_row, dtype=np.int32)
        B = kpr.shape[0]
    n_draft_total = dl.shape[0]
    assert tl.shape[0] == n_draft_total + B
    toks = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    temp = np.ascontiguousarray(temperature, dtype=np.float32).reshape(-1)
    assert temp.shape[0] in (1, B)
    per_row = int(temp.shape[0] == B and B > 1)
    uni = np.ascontiguousarray(uniforms, dtype=np.float32)
    assert uni.shape[0] == n_draft_total + B and toks.shape[0] == n_draft_total

    res = OracleResult(
        accepted_len=np.full(B, -1, np.int32),
        emitted_tokens=np.full(n_draft_total + B, -1, np.int32),
        row_status=np.zeros(B, np.int32),
        p_tok=np.full(n_draft_total, np.nan), q_tok=np.full(n_draft_total, np.nan),
        rho=np.full(n_draft_total, np.nan), accept_margin=np.full(n_draft_total, np.nan),
        cdf_margin=np.full(B, np.nan))

    def run(b0, b1):
        rc = lib.oracle_spec_verify(
            _ptr(tl), _ptr(dl), dtype, V, ld_t, ld_d, _ptr(toks), _ptr(kpr), B, int(k_uniform),
            n_draft_total, _ptr(temp), per_row, _ptr(uni), b0, b1,
            _ptr(res.accepted_len), _ptr(res.emitted_tokens), _ptr(res.row_status),
            _ptr(res.p_tok), _ptr(res.q_tok), _ptr(res.rho), _ptr(res.accept_margin),
            _ptr(res.cdf_margin))
        if rc != 0:
            raise MemoryError("oracle scratch allocation failed")

    lo, hi = (0, B) if b_range is None else b_range
    threads = max(1, min(int(threads), hi - lo))
    if threads == 1:
        run(lo, hi)
    else:
        # contiguous blocks, many more blocks than threads so ragged K balances out
        n_blocks = min(hi - lo, threads * 8)
        edges = np.linspace(lo, hi, n_blocks + 1).astype(int)
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(lambda k: run(int(edges[k]), int(edges[k + 1])), range(n_blocks)))
    return res


def position_distributions(target_row, draft_row, temperature: float):
    """(p, q, r) of one position as float64 arrays; r = max(0, p - q), not normalised."""
    lib = _load()
    dtype = _dtype_code(target_row)
    V = target_row.shape[0]
    tr = np.ascontiguousarray(target_row)
    dr = None if draft_row is None else np.ascontiguousarray(draft_row)
    p = np.empty(V)
    q = np.empty(V) if dr is not None else None
    r = np.empty(V) if dr is not None else None
    rc = lib.oracle_position_distributions(_ptr(tr), _ptr(dr), dtype, V, float(temperature),
                                           _ptr(p), _ptr(q), _ptr(r))
    if rc != 0:
        raise MemoryError("oracle scratch allocation failed")
    return p, q, r


def next_lookahead(k_per_row, accepted_len, k_min: int, k_max: int) -> np.ndarray:
    """Lookahead of the next round per sequence: K+2 after a fully accepted draft, else K-1, clamped."""
    lib = _load()
    k = np.ascontiguousarray(k_per_row, dtype=np.int32)
    a = np.ascontiguousarray(accepted_len, dtype=np.int32)
    out = np.empty_like(k)
    lib.oracle_next_lookahead(_ptr(k), 0, _ptr(a), k.shape[0], int(k_min), int(k_max), _ptr(out))
    return out


@dataclass
class GreedyResult:
    accepted_len: np.ndarray      # int32 [B]
    emitted_tokens: np.ndarray    # int32 [n_draft_total + B], target packing, -1 padded
    row_status: np.ndarray        # int32 [B]
    target_argmax: np.ndarray     # int32 [n_draft_total + B]  argmax of every target row (-1: sequence invalid)


def spec_verify_greedy(target_logits, draft_tokens, k_per_row, *, k_uniform: int = 0,
                       threads: int = 1) -> GreedyResult:
    """Greedy verification (temperature -> 0): accept while the draft token is the target row's argmax.

    Arguments as for ``spec_verify`` (no draft logits, temperature or uniforms).
    """
    lib = _load()
    tl = target_logits
    dtype = _dtype_code(tl)
    V = tl.shape[1]
    elt = tl.dtype.itemsize
    assert tl.strides[1] == elt
    ld_t = tl.strides[0] // elt
    if isinstance(k_per_row, (int, np.integer)):
        B, kpr = int(k_per_row), None
    else:
        kpr = np.ascontiguousarray(k_per_row, dtype=np.int32)
        B = kpr.shape[0]
    n_draft_total = tl.shape[0] - B
    toks = np.ascontiguousarray(draft_tokens, dtype=np.int32)
    assert toks.shape[0] == n_draft_total
    res = GreedyResult(
        accepted_len=np.full(B, -1, np.int32),
        emitted_tokens=np.full(n_draft_total + B, -1, np.int32),
        row_status=np.zeros(B, np.int32),
        target_argmax=np.full(n_draft_total + B, -1, np.int32))

    def run(b0, b1):
        lib.oracle_spec_verify_greedy(
            _ptr(tl), dtype, V, ld_t, _ptr(toks), _ptr(kpr), B, int(k_uniform), n_draft_total, b0, b1,
            _ptr(res.accepted_len), _ptr(res.emitted_tokens), _ptr(res.row_status), _ptr(res.target_argmax))

    threads = max(1, min(int(threads), B))
    if threads == 1:
        run(0, B)
    else:
        edges = np.linspace(0, B, min(B, threads * 8) + 1).astype(int)
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(lambda k: run(int(edges[k]), int(edges[k + 1])), range(len(edges) - 1)))
    return res


@dataclass
class TreeResult:
    accepted_len: np.ndarray      # int32 [B]   nodes on the accepted path
    emitted_tokens: np.ndarray    # int32 [n_node_total + B]
    accepted_nodes: np.ndarray    # int32 [n_node_total + B]  node index of each accepted token, -1 otherwise
    row_status: np.ndarray        # int32 [B]
    p_tok: np.ndarray             # float64 [n_node_total]  p_c(x_j), c the parent's context
    q_tok: np.ndarray             # float64 [n_node_total]
    walk_margin: np.ndarray       # float64 [B]  smallest |u - ratio| over the tests the walk made
    cdf_margin: np.ndarray        # float64 [B]


def spec_verify_tree(target_logits, draft_logits, node_tokens, node_parent, n_per_seq, temperature, uniforms,
                     *, threads: int = 1) -> TreeResult:
    """Tree-structured verification on host arrays (layout: see the C file).  n_per_seq int32 [B]."""
    lib = _load()
    tl, dl = target_logits, draft_logits
    dtype = _dtype_code(tl)
    V = tl.shape[1]
    elt = tl.dtype.itemsize
    assert dl.dtype == tl.dtype and tl.strides[1] == elt and (dl.size == 0 or dl.strides[1] == elt)
    ld_t = tl.strides[0] // elt
    ld_d = dl.strides[0] // elt if dl.shape[0] > 0 else V
    npr = np.ascontiguousarray(n_per_seq, dtype=np.int32)
    B = npr.shape[0]
    n_total = dl.shape[0]
    assert tl.shape[0] == n_total + B
    toks = np.ascontiguousarray(node_tokens, dtype=np.int32)
    par = np.ascontiguousarray(node_parent, dtype=np.int32)
    temp = np.ascontiguousarray(temperature, dtype=np.float32).reshape(-1)
    assert temp.shape[0] in (1, B)
    per_seq = int(temp.shape[0] == B and B > 1)
    uni = np.ascontiguousarray(uniforms, dtype=np.float32)
    assert uni.shape[0] == n_total + B and toks.shape[0] == n_total and par.shape[0] == n_total
    res = TreeResult(
        accepted_len=np.full(B, -1, np.int32), emitted_tokens=np.full(n_total + B, -1, np.int32),
        accepted_nodes=np.full(n_total + B, -1, np.int32), row_status=np.zeros(B, np.int32),
        p_tok=np.full(n_total, np.nan), q_tok=np.full(n_total, np.nan),
        walk_margin=np.full(B, np.nan), cdf_margin=np.full(B, np.nan))

    def run(b0, b1):
        rc = lib.oracle_spec_verify_tree(
            _ptr(tl), _ptr(dl), dtype, V, ld_t, ld_d, _ptr(toks), _ptr(par), _ptr(npr), B, 0, n_total,
            _ptr(temp), per_seq, _ptr(uni), b0, b1, _ptr(res.accepted_len), _ptr(res.emitted_tokens),
            _ptr(res.accepted_nodes), _ptr(res.row_status), _ptr(res.p_tok), _ptr(res.q_tok),
            _ptr(res.walk_margin), _ptr(res.cdf_margin))
        if rc != 0:
            raise MemoryError("oracle scratch allocation failed")

    threads = max(1, min(int(threads), B))
    if threads == 1:
        run(0, B)
    else:
        edges = np.linspace(0, B, min(B, threads * 8) + 1).astype(int)
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(lambda k: run(int(edges[k]), int(edges[k + 1])), range(len(edges) - 1)))
    return res


def lm_head(hidden: np.ndarray, weight: np.ndarray, *, threads: int = 1) -> np.ndarray:
    """logits = hidden @ weight.T for bf16 bit patterns (uint16 arrays [M, H] and [V, H]): products
    summed in double, one rounding to bf16.  Returns uint16 [M, V]."""
    lib = _load()
    h = np.ascontiguousarray(hidden, dtype=np.uint16)
    w = np.ascontiguousarray(weight, dtype=np.uint16)
    M, H = h.shape
    V = w.shape[0]
    assert w.shape[1] == H
    out = np.zeros((M, V), np.uint16)

    def run(r0, r1):
        lib.oracle_lm_head(_ptr(h), H, _ptr(w), H, M, V, H, r0, r1, _ptr(out), V)

    threads = max(1, min(int(threads), M))
    if threads == 1:
        run(0, M)
    else:
        edges = np.linspace(0, M, min(M, threads * 4) + 1).astype(int)
        with ThreadPoolExecutor(max_workers=threads) as pool:
            list(pool.map(lambda k: run(int(edges[k]), int(edges[k + 1])), range(len(edges) - 1)))
    return out
