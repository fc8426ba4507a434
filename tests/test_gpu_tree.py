"""Tree-structured verification on the GPU vs the fp64 oracle, through the C ABI.

Bar (as for the chain): accepted path and emitted tokens identical except where the oracle's own
decision margin is below 1e-5 (|u - ratio| of a test the walk made, or the last uniform's distance
to a CDF step) -- counted; per-node probabilities within 1e-5 relative."""
import numpy as np
import pytest
import torch

import oracle
from gpu_utils import logits_to_torch, ORACLE_THREADS, PROB_RTOL
from helpers import probs_to_logits, f32_to_bf16_bits
from paper_2411_00853_b200 import binding
from paper_2411_00853_b200 import workloads as W

pytestmark = [pytest.mark.gpu, pytest.mark.usefixtures("kernel_path")]


class TreeCase:
    def __init__(self, tl, dl, tok, par, n, T, uni):
        self.target_logits, self.draft_logits, self.draft_tokens, self.node_parent = tl, dl, tok, par
        self.k_per_row, self.temperature, self.uniforms = np.asarray(n, np.int32), T, uni
        self.B, self.V = len(n), tl.shape[1]
        self.off_d = np.concatenate([[0], np.cumsum(np.maximum(self.k_per_row, 0))]).astype(np.int64)
        self.off_t = self.off_d[:-1] + np.arange(self.B)
        self.n_draft_total = dl.shape[0]


def run_gpu(w, ld_pad=0, elem_offset=0):
    D, B, V = w.n_draft_total, w.B, w.V

    def place(a, rows):
        t = logits_to_torch(a)
        ld = V + ld_pad
        buf = torch.full((rows * ld + elem_offset + 16,), float("nan"), dtype=t.dtype, device="cuda")
        view = buf[elem_offset:elem_offset + rows * ld].view(rows, ld)[:, :V]
        if rows:
            view.copy_(t.cuda())
        return buf, view

    _tb, tl = place(w.target_logits, D + B)
    _db, dl = place(w.draft_logits, D)
    i32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.int32)).cuda()
    f32 = lambda a: torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
    acc = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    em = torch.full((D + B,), -7, dtype=torch.int32, device="cuda")
    nodes = torch.full((D + B,), -7, dtype=torch.int32, device="cuda")
    st = torch.full((B,), -7, dtype=torch.int32, device="cuda")
    dp = torch.full((D,), float("nan"), dtype=torch.float32, device="cuda")
    dq = torch.full((D,), float("nan"), dtype=torch.float32, device="cuda")
    binding.spec_verify_tree(tl, dl, i32(w.draft_tokens), i32(w.node_parent), i32(w.k_per_row), f32(w.temperature),
                             f32(w.uniforms), accepted_len=acc, emitted_tokens=em, accepted_nodes=nodes,
                             row_status=st, diag_p_tok=dp, diag_q_tok=dq)
    torch.cuda.synchronize()
    return tuple(t.cpu().numpy() for t in (acc, em, nodes, st, dp, dq))


def run_oracle(w):
    return oracle.spec_verify_tree(w.target_logits, w.draft_logits, w.draft_tokens, w.node_parent, w.k_per_row,
                                   w.temperature, w.uniforms, threads=ORACLE_THREADS)


def assert_tree_parity(w, got, max_excused_frac=0.02):
    acc, em, nodes, st, dp, dq = got
    ora = run_oracle(w)
    bad_bits = 1 | 2 | 4 | 32
    assert np.array_equal(st & bad_bits, ora.row_status & bad_bits), "row_status differs"
    identical = excused = 0
    failures = []
    for b in range(w.B):
        N = max(int(w.k_per_row[b]), 0)
        d0, t0 = int(w.off_d[b]), int(w.off_t[b])
        if ora.row_status[b] & bad_bits:
            assert acc[b] == 0
            if not (ora.row_status[b] & 1):
                assert np.all(em[t0:t0 + N + 1] == -1) and np.all(nodes[t0:t0 + N + 1] == -1)
            continue
        np.testing.assert_allclose(dp[d0:d0 + N], ora.p_tok[d0:d0 + N], rtol=PROB_RTOL, atol=1e-37)
        np.testing.assert_allclose(dq[d0:d0 + N], ora.q_tok[d0:d0 + N], rtol=PROB_RTOL, atol=1e-37)
        sl = slice(t0, t0 + N + 1)
        # the GPU result is a valid walk whatever the oracle says
        a = int(acc[b])
        assert 0 <= a <= N
        prev = -1
        for i in range(a):
            j = int(nodes[t0 + i])
            assert 0 <= j < N and w.node_parent[d0 + j] == prev and em[t0 + i] == w.draft_tokens[d0 + j]
            prev = j
        assert 0 <= em[t0 + a] < w.V and np.all(em[t0 + a + 1:t0 + N + 1] == -1) and np.all(nodes[t0 + a:t0 + N + 1] == -1)
        same = (acc[b] == ora.accepted_len[b] and np.array_equal(em[sl], ora.emitted_tokens[sl])
                and np.array_equal(nodes[sl], ora.accepted_nodes[sl]))
        if same:
            identical += 1
        elif ora.walk_margin[b] < 1e-5 or ora.cdf_margin[b] < 1e-5:
            excused += 1
        else:
            failures.append((b, int(acc[b]), int(ora.accepted_len[b]), float(ora.walk_margin[b]), float(ora.cdf_margin[b])))
    assert not failures, f"{len(failures)} sequences differ from the oracle outside the 1e-5 margin: {failures[:6]}"
    assert excused <= max(1, int(max_excused_frac * w.B)), f"too many thin-margin excuses: {excused}"
    return identical, excused, ora


@pytest.mark.parametrize("V", [1, 2, 7, 9, 33, 257, 1000, 4099, 20000])
@pytest.mark.parametrize("dtype", ["f32", "bf16", "f16"])
def test_small_and_odd_vocabularies(dtype, V):
    w = W.make_tree_config(B=20, V=V, dtype=dtype, seed=V)
    identical, excused, ora = assert_tree_parity(w, run_gpu(w), max_excused_frac=0.1)
    if V >= 257:
        assert ora.accepted_len.max() >= 2


def test_one_cta_and_paired_ctas_give_the_same_walks():
    """A batch of at most half as many sequences as the device has SMs is resolved by a pair of CTAs
    per sequence, a larger one by single CTAs: the first 60 sequences of a batch of 100 (single CTAs) must
    come out exactly as when they are submitted alone (pairs), and both must agree with the oracle."""
    w = W.make_tree_config(B=100, V=6001, dtype="bf16", seed=21)
    got_all = run_gpu(w)
    acc_all, em_all, nodes_all = got_all[:3]
    assert_tree_parity(w, got_all, max_excused_frac=0.05)
    sub = w.take(0, 60)
    acc, em, nodes = run_gpu(sub)[:3]
    n_slots = sub.n_draft_total + sub.B
    assert np.array_equal(acc, acc_all[:60])
    assert np.array_equal(em[:n_slots], em_all[:n_slots])
    assert np.array_equal(nodes[:n_slots], nodes_all[:n_slots])


def test_many_siblings():
    """A root with twelve children drawn from a poor draft: long runs of rejections, each with its
    own pass and coefficient."""
    rng = np.random.default_rng(8)
    B, V, m = 32, 5000, 12
    n = np.full(B, m, np.int32)
    tl = (rng.normal(size=(B * (m + 1), V)) * 3).astype(np.float32)
    dl = np.full((B * m, V), np.nan, np.float32)
    tok = np.empty(B * m, np.int32)
    for b in range(B):
        row = (tl[b * (m + 1)] * 0.3 + rng.normal(size=V) * 2.5).astype(np.float32)
        dl[b * m] = row
        g = rng.gumbel(size=(m, V))
        tok[b * m:(b + 1) * m] = np.argmax(row / 0.9 + g, axis=1)
    par = np.full(B * m, -1, np.int32)
    uni = rng.random(B * (m + 1)).astype(np.float32)
    w = TreeCase(tl, dl, tok, par, n, np.array([0.9], np.float32), uni)
    identical, excused, ora = assert_tree_parity(w, run_gpu(w), max_excused_frac=0.1)
    assert (ora.accepted_len == 0).sum() >= 3 and (ora.accepted_nodes[w.off_t] >= 3).sum() >= 3


def test_hand_cases_on_the_gpu():
    P, Q, ANY = [0.4, 0.3, 0.2, 0.1], [0.1, 0.2, 0.3, 0.4], [0.25] * 4
    lg = lambda rows: probs_to_logits(np.asarray(rows, np.float64))

    def one(target, draft, tokens, parents, u, u_last):
        N = len(tokens)
        w = TreeCase(lg(target), lg(draft).reshape(N, 4), np.asarray(tokens, np.int32), np.asarray(parents, np.int32),
                     [N], np.array([1.0], np.float32), np.asarray(list(u) + [u_last], np.float32))
        acc, em, nodes, st, dp, dq = run_gpu(w)
        return int(acc[0]), em[:acc[0] + 1].tolist(), nodes[:acc[0]].tolist()
    # second child accepted after the first is rejected (residual (0.75, 0.25, 0, 0), ratio 1.25)
    assert one([P, ANY, [1e-30, 1e-30, 1, 1e-30]], [Q, ANY], [3, 1], [-1, -1], [0.5, 0.99], 0.3) == (1, [1, 2], [1])
    # both rejected: r = (13/14, 1/14, 0, 0)
    assert one([P, ANY, ANY], [Q, ANY], [3, 2], [-1, -1], [0.5, 0.0], 0.9) == (0, [0], [])
    assert one([P, ANY, ANY], [Q, ANY], [3, 2], [-1, -1], [0.5, 0.0], 0.95) == (0, [1], [])
    # first child accepted, its only child rejected, residual (0, 0, 0.25, 0.75)
    assert one([P, Q, ANY, ANY], [Q, P, ANY], [3, 1, 0], [-1, -1, 0], [0.2, 0.0, 0.3], 0.2) == (1, [3, 2], [0])


def test_chains_agree_with_the_chain_entry_point():
    w5 = W.make_config(5, B=40, V=3001)
    par = np.concatenate([np.arange(-1, K - 1) for K in w5.k_per_row]).astype(np.int32)
    w = TreeCase(w5.target_logits, w5.draft_logits, w5.draft_tokens, par, w5.k_per_row, w5.temperature, w5.uniforms)
    identical, excused, ora = assert_tree_parity(w, run_gpu(w))
    chain = oracle.spec_verify(w5.target_logits, w5.draft_logits, w5.draft_tokens, w5.k_per_row, w5.temperature,
                               w5.uniforms)
    assert np.array_equal(ora.emitted_tokens, chain.emitted_tokens)


@pytest.mark.parametrize("ld_pad,elem_offset", [(0, 1), (3, 0), (5, 3), (8, 8)])
def test_unaligned_rows_and_padded_pitch(ld_pad, elem_offset):
    w = W.make_tree_config(B=6, V=3001, dtype="bf16", seed=3)
    ref = run_gpu(w)
    got = run_gpu(w, ld_pad=ld_pad, elem_offset=elem_offset)
    assert_tree_parity(w, got)
    assert all(np.array_equal(a, b) for a, b in zip(ref[:4], got[:4]))


def test_data_errors_never_fault():
    w = W.make_tree_config(B=10, V=1200, dtype="bf16", seed=9)
    par = w.node_parent.copy()
    tok = w.draft_tokens.copy()
    n = w.k_per_row.copy()
    par[int(w.off_d[1]) + 2] = 2            # own index
    par[int(w.off_d[2]) + 1] = -5
    par[int(w.off_d[3]) + 1] = 1 << 30
    tok[int(w.off_d[4])] = -1
    bad = TreeCase(w.target_logits, w.draft_logits, tok, par, n, w.temperature, w.uniforms)
    got = run_gpu(bad)
    identical, excused, ora = assert_tree_parity(bad, got)
    assert ora.row_status[1:5].tolist() == [32, 32, 32, 4] and not ora.row_status[5:].any()
    # node counts that overrun the buffers, and a negative one
    n2 = w.k_per_row.copy(); n2[9] += 3
    assert_tree_parity(TreeCase(w.target_logits, w.draft_logits, w.draft_tokens, w.node_parent, n2, w.temperature,
                                w.uniforms), run_gpu(TreeCase(w.target_logits, w.draft_logits, w.draft_tokens,
                                                              w.node_parent, n2, w.temperature, w.uniforms)))
    T = np.array([0.0], np.float32)
    got = run_gpu(TreeCase(w.target_logits, w.draft_logits, w.draft_tokens, w.node_parent, w.k_per_row, T, w.uniforms))
    assert np.all(got[3] == 2) and np.all(got[0] == 0) and np.all(got[1] == -1)


def test_full_size_tree_batch():
    w = W.make_tree_config()                 # B=64, V=128256, bf16
    identical, excused, ora = assert_tree_parity(w, run_gpu(w))
    print(f"tree batch: {identical} identical, {excused} excused; mean accepted {ora.accepted_len.mean():.2f}; "
          f"{w.n_draft_total} nodes, {w.n_internal} contexts with children")
    assert identical + excused == w.B
