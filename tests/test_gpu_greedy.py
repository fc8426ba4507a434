"""Greedy verification on the GPU vs the oracle: integer work, so everything is compared for
exact equality -- accepted lengths, emitted tokens, row status and the argmax of every row."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import logits_to_torch
from helpers import f32_to_bf16_bits
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("kernel_path")]


def _to_device(a, ld_pad=0, elem_offset=0):
    t = logits_to_torch(a)
    rows, V = t.shape
    ld = V + ld_pad
    buf = torch.full((rows * ld + elem_offset + 16,), float("nan"), dtype=t.dtype, device="cuda")
    view = buf[elem_offset:elem_offset + rows * ld].view(rows, ld)[:, :V]
    view.copy_(t.cuda())
    return buf, view


def run_gpu(target, tokens, k, **place):
    buf, tl = _to_device(target, **place)
    B, D = len(k), len(tokens)
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    em = torch.full((D + B,), -7, dtype=torch.int32, device="cuda")
    st = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    am = torch.full((D + B,), -7, dtype=torch.int32, device="cuda")
    binding.spec_verify_greedy(tl, torch.from_numpy(np.ascontiguousarray(tokens)).cuda(),
                               torch.from_numpy(np.ascontiguousarray(k)).cuda(),
                               accepted_len=acc, emitted_tokens=em, row_status=st, target_argmax=am)
    torch.cuda.synchronize()
    return acc.cpu().numpy(), em.cpu().numpy(), st.cpu().numpy(), am.cpu().numpy()


def assert_equal_to_oracle(target, tokens, k, got):
    ora = oracle.spec_verify_greedy(target, tokens, k, threads=16)
    acc, em, st, am = got
    assert np.array_equal(st, ora.row_status)
    assert np.array_equal(acc, ora.accepted_len)
    assert np.array_equal(em, ora.emitted_tokens)
    valid = ora.target_argmax >= 0
    assert np.array_equal(am[valid], ora.target_argmax[valid])
    return ora


def greedy_tokens(w, rng, p_match=0.8):
    """Draft tokens for a greedy run on workload w: the target row's argmax with probability
    p_match, else the workload's own (sampled) draft token."""
    best = oracle.spec_verify_greedy(w.target_logits, w.draft_tokens, w.k_per_row, threads=16).target_argmax
    tok = w.draft_tokens.copy()
    for b in range(w.B):
        for i in range(int(w.k_per_row[b])):
            if rng.random() < p_match:
                tok[w.off_d[b] + i] = best[w.off_t[b] + i]
    return tok


@pytest.mark.parametrize("V", [1, 2, 7, 8, 9, 33, 257, 1000, 4099, 20000])
@pytest.mark.parametrize("cfg", [1, 2, 5])
def test_small_and_odd_vocabularies(cfg, V):
    w = W.make_config(cfg, B=24, V=V)
    tok = greedy_tokens(w, np.random.default_rng(V))
    ora = assert_equal_to_oracle(w.target_logits, tok, w.k_per_row, run_gpu(w.target_logits, tok, w.k_per_row))
    if V > 100:
        assert 0 < ora.accepted_len.sum() < w.k_per_row.sum()


@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_ties_everywhere(dtype):
    """Rows drawn from thirteen values: every row has many equal maxima, spread over lanes, warps,
    chunks; the smallest token id must win."""
    rng = np.random.default_rng(17)
    B, V = 70, 40000 if dtype == "f32" else 70000
    k = rng.integers(0, 4, B).astype(np.int32)
    D = int(k.sum())
    grid = rng.integers(-6, 7, (D + B, V)).astype(np.float32) * 0.5
    grid[:, : V // 2] -= 0.5 * (rng.random((D + B, 1)) < 0.5)      # half the rows: maxima only in the upper half
    target = {"f32": grid, "bf16": f32_to_bf16_bits(grid), "f16": grid.astype(np.float16)}[dtype]
    tok = rng.integers(0, V, D).astype(np.int32)
    got = run_gpu(target, tok, k)
    assert_equal_to_oracle(target, tok, k, got)
    assert np.array_equal(got[3], np.argmax(grid, axis=1))


@pytest.mark.parametrize("ld_pad,elem_offset", [(0, 1), (3, 0), (5, 3), (8, 8)])
def test_unaligned_rows_and_padded_pitch(ld_pad, elem_offset):
    w = W.make_config(5, B=6, V=3001)
    tok = greedy_tokens(w, np.random.default_rng(1))
    got = run_gpu(w.target_logits, tok, w.k_per_row, ld_pad=ld_pad, elem_offset=elem_offset)
    assert_equal_to_oracle(w.target_logits, tok, w.k_per_row, got)


def test_special_values():
    V = 5000
    t = np.random.default_rng(2).normal(size=(6, V)).astype(np.float32)
    t[0, :] = -np.inf                      # nothing above -inf -> token 0
    t[1, 17] = np.nan; t[1, 4000] = 50.0   # NaN is never the largest
    t[2, :] = 0.0; t[2, 9] = -0.0          # +0 and -0 are equal: token 0
    t[3, V - 1] = 99.0                     # last element
    t[4, 0] = 99.0                         # first element
    k = np.zeros(6, np.int32)
    got = run_gpu(t, np.zeros(0, np.int32), k)
    assert_equal_to_oracle(t, np.zeros(0, np.int32), k, got)
    assert got[1][:5].tolist() == [0, 4000, 0, V - 1, 0]


def test_data_errors_and_uniform_k():
    w = W.make_config(2, B=8, V=2000)
    tok = greedy_tokens(w, np.random.default_rng(4))
    tok[int(w.off_d[3])] = w.V             # out of range
    k = w.k_per_row.copy()
    k[5] = -2                              # shifts the packing of later sequences; still no fault
    got = run_gpu(w.target_logits, tok, k)
    ora = assert_equal_to_oracle(w.target_logits, tok, k, got)
    assert ora.row_status[5] == oracle.ROW_BAD_K and (ora.row_status != 0).sum() >= 2
    # k_per_row == NULL with k_uniform
    tok = greedy_tokens(w, np.random.default_rng(5))
    _, tl = _to_device(w.target_logits)
    acc, em = binding.spec_verify_greedy(tl, torch.from_numpy(tok).cuda(), None, k_uniform=int(w.k_per_row[0]))
    ora = oracle.spec_verify_greedy(w.target_logits, tok, w.k_per_row)
    assert np.array_equal(acc.cpu().numpy(), ora.accepted_len) and np.array_equal(em.cpu().numpy(), ora.emitted_tokens)


def test_argument_errors():
    lib = binding.load()
    t = torch.zeros(4, 64, device="cuda")
    ws = torch.empty(4096, dtype=torch.uint8, device="cuda")
    out = torch.empty(8, dtype=torch.int32, device="cuda")
    tok = torch.zeros(3, dtype=torch.int32, device="cuda")

    def call(dtype=0, V=64, ld=64, B=1, k=3, D=3, target=t, ws_bytes=4096):
        return lib.spec_verify_greedy(target.data_ptr() if target is not None else None, dtype, V, ld, tok.data_ptr(),
                                      None, B, k, D, out.data_ptr(), out.data_ptr(), None, None, ws.data_ptr(),
                                      ws_bytes, None, binding.default_flags() & 3)
    assert call() == 0
    assert call(dtype=3) == 3 and call(ld=63) == 2 and call(k=2) == 2 and call(target=None) == 1
    assert call(ws_bytes=16) == 5
    torch.cuda.synchronize()


@pytest.mark.parametrize("cfg", [3, 5])
def test_large_config_full_size(cfg):
    w = W.make_config(cfg)
    tok = greedy_tokens(w, np.random.default_rng(cfg))
    got = run_gpu(w.target_logits, tok, w.k_per_row)
    ora = assert_equal_to_oracle(w.target_logits, tok, w.k_per_row, got)
    assert 0 < ora.accepted_len.sum() < w.k_per_row.sum()
